"""ctypes binding of liblibra.so: the same entry points as include/libra.h, argument
marshalling only.  Tensors are torch CUDA tensors (device memory and streams come from
torch); every computation runs in the library's kernels.

Importing this module loads the library and raises if it has not been built — there is
no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "liblibra.so")
if not os.path.exists(_SO):
    raise ImportError(f"{_SO} is missing: run `python -m paper_2607_23250_b200.build` (needs nvcc)")
_lib = ctypes.CDLL(_SO)

LIBRA_DIR_Q, LIBRA_DIR_KV, LIBRA_DIR_PAIR = 1, 2, 4
LIBRA_WEIGHT_PAIRS, LIBRA_WEIGHT_BLOCKS = 0, 1
KERNEL_FWD, KERNEL_BWD_DKDV, KERNEL_BWD_DQ, KERNEL_BWD_PREP, KERNEL_BWD_FUSED, KERNEL_BWD_POST = 1, 2, 3, 4, 5, 6
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_PLAN_MISMATCH, ERR_CUDA = -1, -2, -3, -4
ERR_OVERFLOW, ERR_TIMEOUT, ERR_BAD_SEQLENS, ERR_NO_DEVICE = -5, -6, -7, -8
ERR_SCRATCH_TOO_SMALL = -9

EXPORTS = ["libra_plan_tiles", "libra_plan_info", "libra_plan_status", "libra_plan_export",
           "libra_plan_export_pairs", "libra_plan_destroy", "libra_attn_pool_fwd", "libra_attn_pool_bwd_workspace_bytes",
           "libra_attn_pool_bwd", "libra_attn_pool_bwd_noalloc_max_bytes", "libra_attn_pool_bwd_noalloc",
           "libra_tap_schedule", "libra_busy_times", "libra_tile_times", "libra_plan_set_wait_limit_ns", "libra_plan_inject_stall", "libra_plan_set_timing", "libra_kernel_time_ms", "libra_kernel_times_ms", "libra_selftest_wait_timeout", "libra_launch_count",
           "libra_strerror"]


class PlanOpts(ctypes.Structure):
    _fields_ = [("n_workers", ctypes.c_int), ("directions", ctypes.c_int), ("tile_kv", ctypes.c_int),
                ("n_heads_kv", ctypes.c_int), ("total_tokens", ctypes.c_int64), ("weight_model", ctypes.c_int),
                ("cost_block", ctypes.c_int), ("unit_cost_q", ctypes.c_int), ("unit_cost_kv", ctypes.c_int),
                ("pair_chunk", ctypes.c_int)]


class Dims(ctypes.Structure):
    _fields_ = [("total_tokens", ctypes.c_int64), ("n_samples", ctypes.c_int), ("hq", ctypes.c_int),
                ("hkv", ctypes.c_int), ("head_dim", ctypes.c_int), ("softmax_scale", ctypes.c_float)]


_lib.libra_strerror.restype = ctypes.c_char_p
_lib.libra_launch_count.restype = ctypes.c_int64
_lib.libra_attn_pool_bwd_workspace_bytes.restype = ctypes.c_size_t
_lib.libra_attn_pool_bwd_noalloc_max_bytes.restype = ctypes.c_size_t
_vp = ctypes.c_void_p


class LibraError(RuntimeError):
    def __init__(self, code, what):
        self.code = code
        super().__init__(f"{what}: {_lib.libra_strerror(code).decode()} ({code})")


def _check(code, what):
    if code != 0:
        raise LibraError(code, what)


def _ptr(t):
    return _vp(t.data_ptr()) if t is not None else _vp(0)


def _np(a):
    return a.ctypes.data_as(_vp) if a is not None else _vp(0)


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return _vp(s.cuda_stream)


def libra_selftest_wait_timeout(limit_ns: int):
    """(status, nanoseconds waited) of a wait on a barrier nothing arrives on; status is ERR_TIMEOUT by design."""
    st, ns = ctypes.c_int(), ctypes.c_int()
    _check(_lib.libra_selftest_wait_timeout(ctypes.c_uint32(limit_ns), ctypes.byref(st), ctypes.byref(ns)),
           "libra_selftest_wait_timeout")
    return st.value, ns.value


def launch_count() -> int:
    return int(_lib.libra_launch_count())


class Plan:
    """Owner of a libra_plan_t."""

    def __init__(self, handle, cu_seqlens):
        self._h = handle
        self.cu_seqlens = cu_seqlens  # kept alive for the attention calls

    def info(self, direction=LIBRA_DIR_Q):
        nt, nb = ctypes.c_int64(), ctypes.c_int64()
        w, tile, h = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
        _check(_lib.libra_plan_info(self._h, direction, ctypes.byref(nt), ctypes.byref(w), ctypes.byref(nb),
                                    ctypes.byref(tile), ctypes.byref(h)), "libra_plan_info")
        return dict(n_tiles=nt.value, n_workers=w.value, n_blocks=nb.value, tile=tile.value, n_heads=h.value)

    def status(self) -> int:
        return int(_lib.libra_plan_status(self._h))

    def export(self, direction=LIBRA_DIR_Q):
        i = self.info(direction)
        nt, w = i["n_tiles"], i["n_workers"]
        res = dict(weight=np.empty(nt, np.int64), order=np.empty(nt, np.int32), cta_of_tile=np.empty(nt, np.int32),
                   cta_offsets=np.empty(w + 1, np.int32), cta_tiles=np.empty(nt, np.int32),
                   loads=np.empty(w, np.int64))
        _check(_lib.libra_plan_export(self._h, direction, _np(res["weight"]), _np(res["order"]),
                                      _np(res["cta_of_tile"]), _np(res["cta_offsets"]), _np(res["cta_tiles"]),
                                      _np(res["loads"])), "libra_plan_export")
        res["n_blocks"] = i["n_blocks"]
        return res

    def export_pairs(self):
        """(key_block, query_chunk) of every pair-block and the chunk size in tokens (LIBRA_DIR_PAIR plans)."""
        nb = self.info(LIBRA_DIR_PAIR)["n_blocks"]
        kb, qc, chunk = np.empty(nb, np.int32), np.empty(nb, np.int32), ctypes.c_int()
        _check(_lib.libra_plan_export_pairs(self._h, _np(kb), _np(qc), ctypes.byref(chunk)), "libra_plan_export_pairs")
        return kb, qc, chunk.value

    def busy_times(self, which=KERNEL_FWD):
        w = self.info(LIBRA_DIR_PAIR if which == KERNEL_BWD_FUSED else
                      (LIBRA_DIR_KV if which == KERNEL_BWD_DKDV else LIBRA_DIR_Q))["n_workers"]
        out = np.zeros(w, np.uint64)
        _check(_lib.libra_busy_times(self._h, which, _np(out)), "libra_busy_times")
        return out

    def set_wait_limit_ns(self, ns: int):
        _check(_lib.libra_plan_set_wait_limit_ns(self._h, ctypes.c_uint64(ns)), "libra_plan_set_wait_limit_ns")

    def inject_stall(self, enabled=True):
        _check(_lib.libra_plan_inject_stall(self._h, 1 if enabled else 0), "libra_plan_inject_stall")

    def set_timing(self, enabled=True):
        _check(_lib.libra_plan_set_timing(self._h, 1 if enabled else 0), "libra_plan_set_timing")

    def kernel_time_ms(self, which=KERNEL_FWD) -> float:
        ms = ctypes.c_float()
        _check(_lib.libra_kernel_time_ms(self._h, which, ctypes.byref(ms)), "libra_kernel_time_ms")
        return float(ms.value)

    def tile_times(self, which=KERNEL_FWD):
        """Nanoseconds each tile took in the last launch of the forward (query-major tiles) or the fused backward
        (pair tiles), indexed by tile id (uint32 numpy array)."""
        nt = self.info(LIBRA_DIR_PAIR if which == KERNEL_BWD_FUSED else LIBRA_DIR_Q)["n_tiles"]
        out = np.zeros(nt, dtype=np.uint32)
        _check(_lib.libra_tile_times(self._h, which, _np(out)), "libra_tile_times")
        return out

    def kernel_times_ms(self, which=KERNEL_FWD, capacity=64):
        """Durations (ms) of the most recent recorded launches of kernel `which`, oldest first."""
        buf = (ctypes.c_float * capacity)()
        n = ctypes.c_int()
        _check(_lib.libra_kernel_times_ms(self._h, which, buf, ctypes.c_int(capacity), ctypes.byref(n)),
               "libra_kernel_times_ms")
        return [float(buf[i]) for i in range(n.value)]

    def destroy(self):
        if self._h:
            _lib.libra_plan_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def libra_plan_tiles(cu_seqlens: torch.Tensor, n_heads: int, tile_q: int, n_workers: int = 0,
                     directions: int = 0, tile_kv: int = 0, n_heads_kv: int = 0, total_tokens: int = 0,
                     stream=None, weight_model: int = 0, cost_block: int = 0, unit_cost_q: int = 0,
                     unit_cost_kv: int = 0, pair_chunk: int = 0) -> Plan:
    assert cu_seqlens.is_cuda and cu_seqlens.dtype == torch.int32 and cu_seqlens.is_contiguous()
    opts = PlanOpts(n_workers, directions, tile_kv, n_heads_kv, total_tokens, weight_model, cost_block,
                    unit_cost_q, unit_cost_kv, pair_chunk)
    h = _vp()
    _check(_lib.libra_plan_tiles(_ptr(cu_seqlens), ctypes.c_int(cu_seqlens.numel() - 1), ctypes.c_int(n_heads),
                                 ctypes.c_int(tile_q), ctypes.byref(opts), _stream(stream), ctypes.byref(h)),
           "libra_plan_tiles")
    return Plan(h, cu_seqlens)


def _dims(q, k, plan, scale):
    T, hq, d = q.shape
    return Dims(T, plan.cu_seqlens.numel() - 1, hq, k.shape[1], d, 0.0 if scale is None else float(scale))


def _chk(*ts):
    for t in ts:
        assert t.is_cuda and t.is_contiguous(), "expected contiguous CUDA tensors"


def libra_attn_pool_fwd(q, k, v, plan: Plan, out=None, lse=None, scale=None, stream=None):
    """out [T,Hq,d] bf16, lse [Hq,T] fp32 (allocated with torch when not given)."""
    _chk(q, k, v)
    assert q.dtype == k.dtype == v.dtype == torch.bfloat16
    T, hq, d = q.shape
    out = torch.empty_like(q) if out is None else out
    lse = torch.empty((hq, T), dtype=torch.float32, device=q.device) if lse is None else lse
    dims = _dims(q, k, plan, scale)
    _check(_lib.libra_attn_pool_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(plan.cu_seqlens), plan._h, _ptr(out), _ptr(lse),
                                    ctypes.byref(dims), _stream(stream)), "libra_attn_pool_fwd")
    return out, lse


def libra_attn_pool_bwd_workspace_bytes(plan: Plan, q, k) -> int:
    dims = _dims(q, k, plan, None)
    return int(_lib.libra_attn_pool_bwd_workspace_bytes(plan._h, ctypes.byref(dims)))


def libra_attn_pool_bwd(q, k, v, out, lse, dout, plan: Plan, dq=None, dk=None, dv=None, workspace=None,
                        scale=None, stream=None):
    _chk(q, k, v, out, lse, dout)
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(k) if dk is None else dk
    dv = torch.empty_like(v) if dv is None else dv
    if workspace is None:
        workspace = torch.empty(libra_attn_pool_bwd_workspace_bytes(plan, q, k), dtype=torch.uint8, device=q.device)
    dims = _dims(q, k, plan, scale)
    _check(_lib.libra_attn_pool_bwd(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), _ptr(dout),
                                    _ptr(plan.cu_seqlens), plan._h, _ptr(dq), _ptr(dk), _ptr(dv), _ptr(workspace),
                                    ctypes.byref(dims), _stream(stream)), "libra_attn_pool_bwd")
    return dq, dk, dv


def libra_attn_pool_bwd_noalloc_max_bytes() -> int:
    return int(_lib.libra_attn_pool_bwd_noalloc_max_bytes())


def libra_attn_pool_bwd_noalloc(q, k, v, out, lse, dout, plan: Plan, dq, dk, dv, scale=None, stream=None):
    """Backward that takes no workspace and allocates nothing: dq, dk, dv must be passed in.
    Raises LibraError(ERR_SCRATCH_TOO_SMALL) when the pool exceeds the library's built-in scratch."""
    _chk(q, k, v, out, lse, dout, dq, dk, dv)
    dims = _dims(q, k, plan, scale)
    _check(_lib.libra_attn_pool_bwd_noalloc(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(lse), _ptr(dout),
                                            _ptr(plan.cu_seqlens), plan._h, _ptr(dq), _ptr(dk), _ptr(dv),
                                            ctypes.byref(dims), _stream(stream)), "libra_attn_pool_bwd_noalloc")
    return dq, dk, dv


def libra_vrsp_work(sample_offsets: torch.Tensor, seq_first_sample: torch.Tensor, stream=None) -> torch.Tensor:
    """F_i = sum of squared raw-sample lengths of packed sequence i (int64, on the device)."""
    for t in (sample_offsets, seq_first_sample):
        assert t.is_cuda and t.dtype == torch.int32 and t.is_contiguous()
    D = seq_first_sample.numel() - 1
    work = torch.empty(D, dtype=torch.int64, device=sample_offsets.device)
    _check(_lib.libra_vrsp_work(_ptr(sample_offsets), _ptr(seq_first_sample), ctypes.c_int(D), _ptr(work),
                                _stream(stream)), "libra_vrsp_work")
    return work


def libra_vrsp_place(work: torch.Tensor, pool_size: int, stream=None):
    """Algorithm 1 on the device -> dict(order, pool_of_seq, pool_load) of device tensors."""
    assert work.is_cuda and work.dtype == torch.int64 and work.is_contiguous()
    D = work.numel()
    dev = work.device
    order = torch.empty(D, dtype=torch.int32, device=dev)
    pool_of_seq = torch.empty(D, dtype=torch.int32, device=dev)
    pool_load = torch.empty(max(D // max(pool_size, 1), 1), dtype=torch.int64, device=dev)
    scratch = torch.empty(D, dtype=torch.int32, device=dev)
    _check(_lib.libra_vrsp_place(_ptr(work), ctypes.c_int(D), ctypes.c_int(pool_size), _ptr(order), _ptr(pool_of_seq),
                                 _ptr(pool_load), _ptr(scratch), _stream(stream)), "libra_vrsp_place")
    return dict(order=order, pool_of_seq=pool_of_seq, pool_load=pool_load)


class TapOpts(ctypes.Structure):
    _fields_ = [("cp", ctypes.c_int), ("block", ctypes.c_int), ("n_shards", ctypes.c_int), ("hq", ctypes.c_int),
                ("hkv", ctypes.c_int), ("head_dim", ctypes.c_int), ("tau_num", ctypes.c_int), ("tau_den", ctypes.c_int)]


_lib.libra_tap_num_tiles.restype = ctypes.c_int64


def libra_tap_plan(cu_seqlens: torch.Tensor, seq_offsets, cp: int, block: int, n_shards: int, hq: int, hkv: int,
                   head_dim: int, tau_num: int = 3, tau_den: int = 100, stream=None):
    """Tiles, Algorithm 2 and the exchange volumes of one pool -> dict of device tensors
    (sigma, loads, fwd_bytes [W, W], bwd_bytes [W, W], comm_total, status)."""
    assert cu_seqlens.is_cuda and cu_seqlens.dtype == torch.int32 and cu_seqlens.is_contiguous()
    so = (ctypes.c_int32 * len(seq_offsets))(*[int(x) for x in seq_offsets])
    P = len(seq_offsets) - 1
    W = P * cp
    NT = int(_lib.libra_tap_num_tiles(so, ctypes.c_int(P), ctypes.c_int(block), ctypes.c_int(n_shards)))
    if NT <= 0:
        raise RuntimeError("libra_tap_num_tiles: bad arguments")
    dev = cu_seqlens.device
    out = dict(sigma=torch.empty(NT, dtype=torch.int32, device=dev), loads=torch.empty(W, dtype=torch.int64, device=dev),
               fwd_bytes=torch.empty((W, W), dtype=torch.int64, device=dev),
               bwd_bytes=torch.empty((W, W), dtype=torch.int64, device=dev),
               comm_total=torch.empty(1, dtype=torch.int64, device=dev), status=torch.empty(1, dtype=torch.int32, device=dev))
    opts = TapOpts(cp, block, n_shards, hq, hkv, head_dim, tau_num, tau_den)
    _check(_lib.libra_tap_plan(_ptr(cu_seqlens), ctypes.c_int(cu_seqlens.numel() - 1), so, ctypes.c_int(P),
                               ctypes.byref(opts), _ptr(out["sigma"]), _ptr(out["loads"]), _ptr(out["fwd_bytes"]),
                               _ptr(out["bwd_bytes"]), _ptr(out["comm_total"]), _ptr(out["status"]), _stream(stream)),
           "libra_tap_plan")
    return out


def libra_tap_schedule(cu_seqlens: torch.Tensor, seq_offsets, sigma: torch.Tensor, cp: int, block: int, n_shards: int,
                       hq: int, hkv: int, head_dim: int, capacity: int = 0, stream=None) -> torch.Tensor:
    """Transfer records [n, 6] (kind, src, dst, tok0, ntok, shard) implied by assignment `sigma` (device int32).
    Two calls when `capacity` is 0: the first only counts."""
    assert cu_seqlens.is_cuda and cu_seqlens.dtype == torch.int32 and sigma.is_cuda and sigma.dtype == torch.int32
    so = (ctypes.c_int32 * len(seq_offsets))(*[int(x) for x in seq_offsets])
    P = len(seq_offsets) - 1
    opts = TapOpts(cp, block, n_shards, hq, hkv, head_dim, 3, 100)
    dev = cu_seqlens.device
    n = torch.zeros(1, dtype=torch.int64, device=dev)

    def call(cap):
        rec = torch.empty((max(cap, 1), 6), dtype=torch.int32, device=dev)
        _check(_lib.libra_tap_schedule(_ptr(cu_seqlens), ctypes.c_int(cu_seqlens.numel() - 1), so, ctypes.c_int(P),
                                       ctypes.byref(opts), _ptr(sigma), _ptr(rec), ctypes.c_int64(cap), _ptr(n),
                                       _stream(stream)), "libra_tap_schedule")
        return rec

    if capacity <= 0:
        call(0)
        capacity = int(n.item())
    rec = call(capacity)
    return rec[:min(capacity, int(n.item()))]
