"""ctypes front end of the CPU oracle (oracle.c).

TEST INFRASTRUCTURE ONLY.  Imported by tests, by the smoke check and by the
benchmark's CPU-baseline leg; the product package never imports it.  Inputs and
outputs are numpy arrays; fp32 entry points take float32, fp64 ones take float64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "liboracle.so")
_SRC = [os.path.join(_HERE, "oracle.c"), os.path.join(_HERE, "oracle_attn.inc")]
_lib = None


def build(force: bool = False) -> str:
    """Compile oracle.c into liboracle.so next to it (gcc, OpenMP, no fast-math)."""
    stale = force or not os.path.exists(_SO) or any(
        os.path.getmtime(s) > os.path.getmtime(_SO) for s in _SRC)
    if stale:
        tmp = _SO + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O3", "-march=native", "-fopenmp", "-shared", "-fPIC",
                               "-std=c11", _SRC[0], "-o", tmp, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_SO)
        _lib.oracle_plan_num_blocks.restype = ctypes.c_int64
    return _lib


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def _real(prec):
    return {"f32": np.float32, "f64": np.float64}[prec]


def _arr(x, dt):
    return np.ascontiguousarray(np.asarray(x), dtype=dt)


def _check(rc, what):
    if rc != 0:
        raise RuntimeError(f"{what} failed with code {rc}")


def attn_fwd(q, k, v, cu, scale=None, prec="f32"):
    """Full forward.  q [T,Hq,d], k/v [T,Hkv,d] -> (out [T,Hq,d], lse [Hq,T])."""
    dt = _real(prec)
    q, k, v = _arr(q, dt), _arr(k, dt), _arr(v, dt)
    cu = _arr(cu, np.int32)
    T, hq, d = q.shape
    hkv = k.shape[1]
    assert cu[-1] == T and k.shape == v.shape == (T, hkv, d)
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    out = np.empty_like(q)
    lse = np.empty((hq, T), dtype=dt)
    fn = getattr(_load(), f"oracle_attn_fwd_{prec}")
    _check(fn(_p(q), _p(k), _p(v), _p(cu), ctypes.c_int(len(cu) - 1), ctypes.c_int(hq),
              ctypes.c_int(hkv), ctypes.c_int(d), ctypes.c_double(scale), _p(out), _p(lse)),
           "oracle_attn_fwd")
    return out, lse


def attn_bwd(q, k, v, out, lse, dout, cu, scale=None, prec="f32"):
    """Full backward from the given out/lse -> (dq, dk, dv)."""
    dt = _real(prec)
    q, k, v, out, lse, dout = (_arr(x, dt) for x in (q, k, v, out, lse, dout))
    cu = _arr(cu, np.int32)
    T, hq, d = q.shape
    hkv = k.shape[1]
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    dq, dk, dv = np.empty_like(q), np.empty_like(k), np.empty_like(v)
    fn = getattr(_load(), f"oracle_attn_bwd_{prec}")
    _check(fn(_p(q), _p(k), _p(v), _p(out), _p(lse), _p(dout), _p(cu), ctypes.c_int(len(cu) - 1),
              ctypes.c_int(hq), ctypes.c_int(hkv), ctypes.c_int(d), ctypes.c_double(scale),
              _p(dq), _p(dk), _p(dv)), "oracle_attn_bwd")
    return dq, dk, dv


def attn_fwd_rows(q, k, v, cu, rows, heads, scale=None, prec="f32"):
    """Forward of selected (global row, q head) pairs -> (out_rows [nr,d], lse_rows [nr])."""
    dt = _real(prec)
    q, k, v = _arr(q, dt), _arr(k, dt), _arr(v, dt)
    cu, rows, heads = _arr(cu, np.int32), _arr(rows, np.int64), _arr(heads, np.int32)
    T, hq, d = q.shape
    hkv = k.shape[1]
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    out = np.empty((len(rows), d), dtype=dt)
    lse = np.empty(len(rows), dtype=dt)
    fn = getattr(_load(), f"oracle_attn_fwd_rows_{prec}")
    _check(fn(_p(q), _p(k), _p(v), _p(cu), ctypes.c_int(len(cu) - 1), ctypes.c_int(hq),
              ctypes.c_int(hkv), ctypes.c_int(d), ctypes.c_double(scale), ctypes.c_int(len(rows)),
              _p(rows), _p(heads), _p(out), _p(lse)), "oracle_attn_fwd_rows")
    return out, lse


def attn_dq_rows(q, k, v, dout, cu, rows, heads, scale=None, prec="f32"):
    """dQ of selected (global row, q head) pairs (O and LSE recomputed inside) -> [nr,d]."""
    dt = _real(prec)
    q, k, v, dout = (_arr(x, dt) for x in (q, k, v, dout))
    cu, rows, heads = _arr(cu, np.int32), _arr(rows, np.int64), _arr(heads, np.int32)
    T, hq, d = q.shape
    hkv = k.shape[1]
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    dq = np.empty((len(rows), d), dtype=dt)
    fn = getattr(_load(), f"oracle_attn_dq_rows_{prec}")
    _check(fn(_p(q), _p(k), _p(v), _p(dout), _p(cu), ctypes.c_int(len(cu) - 1), ctypes.c_int(hq),
              ctypes.c_int(hkv), ctypes.c_int(d), ctypes.c_double(scale), ctypes.c_int(len(rows)),
              _p(rows), _p(heads), _p(dq)), "oracle_attn_dq_rows")
    return dq


def attn_dkv_cols(q, k, v, out, lse, dout, cu, cols, kvheads, scale=None, prec="f32"):
    """dK, dV of selected (global key column, kv head) pairs from the given out/lse."""
    dt = _real(prec)
    q, k, v, out, lse, dout = (_arr(x, dt) for x in (q, k, v, out, lse, dout))
    cu, cols, kvheads = _arr(cu, np.int32), _arr(cols, np.int64), _arr(kvheads, np.int32)
    T, hq, d = q.shape
    hkv = k.shape[1]
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    dk = np.empty((len(cols), d), dtype=dt)
    dv = np.empty((len(cols), d), dtype=dt)
    fn = getattr(_load(), f"oracle_attn_dkv_cols_{prec}")
    _check(fn(_p(q), _p(k), _p(v), _p(out), _p(lse), _p(dout), _p(cu), ctypes.c_int(len(cu) - 1),
              ctypes.c_int(hq), ctypes.c_int(hkv), ctypes.c_int(d), ctypes.c_double(scale),
              ctypes.c_int(len(cols)), _p(cols), _p(kvheads), _p(dk), _p(dv)),
           "oracle_attn_dkv_cols")
    return dk, dv


def plan(cu, n_heads, tile, n_workers, direction=0, weight_model=0, cost_block=128, unit_cost=0):
    """SH-Tile plan -> dict(weight, order, cta_of_tile, cta_offsets, cta_tiles, loads).

    weight_model 0: pair count (Eq. 6); 1: block count (cost_block, unit_cost), see oracle_plan_blocks."""
    cu = _arr(cu, np.int32)
    lib = _load()
    n = len(cu) - 1
    nb = lib.oracle_plan_num_blocks(_p(cu), ctypes.c_int(n), ctypes.c_int(tile))
    if nb < 0:
        raise RuntimeError("oracle_plan: bad arguments")
    nt = nb * n_heads
    res = dict(weight=np.empty(nt, np.int64), order=np.empty(nt, np.int32),
               cta_of_tile=np.empty(nt, np.int32), cta_offsets=np.empty(n_workers + 1, np.int32),
               cta_tiles=np.empty(nt, np.int32), loads=np.empty(n_workers, np.int64))
    outs = (_p(res["weight"]), _p(res["order"]), _p(res["cta_of_tile"]), _p(res["cta_offsets"]),
            _p(res["cta_tiles"]), _p(res["loads"]))
    if weight_model == 0:
        _check(lib.oracle_plan(_p(cu), ctypes.c_int(n), ctypes.c_int(n_heads), ctypes.c_int(tile),
                               ctypes.c_int(n_workers), ctypes.c_int(direction), *outs), "oracle_plan")
    else:
        _check(lib.oracle_plan_blocks(_p(cu), ctypes.c_int(n), ctypes.c_int(n_heads), ctypes.c_int(tile),
                                      ctypes.c_int(n_workers), ctypes.c_int(direction), ctypes.c_int(cost_block),
                                      ctypes.c_int(unit_cost), *outs), "oracle_plan_blocks")
    res["n_blocks"] = int(nb)
    return res


def plan_pairs(cu, n_heads, tile, chunk, n_workers):
    """Plan over pair tiles (key block x query chunk x head) -> oracle_plan's dict + key_block, query_chunk per pair-block."""
    cu = _arr(cu, np.int32)
    lib = _load()
    lib.oracle_plan_pairs_num_blocks.restype = ctypes.c_int64
    n = len(cu) - 1
    nu = int(lib.oracle_plan_pairs_num_blocks(_p(cu), ctypes.c_int(n), ctypes.c_int(tile), ctypes.c_int(chunk)))
    if nu < 0:
        raise RuntimeError("oracle_plan_pairs: bad arguments")
    nt = nu * n_heads
    res = dict(weight=np.empty(nt, np.int64), order=np.empty(nt, np.int32), cta_of_tile=np.empty(nt, np.int32),
               cta_offsets=np.empty(n_workers + 1, np.int32), cta_tiles=np.empty(nt, np.int32),
               loads=np.empty(n_workers, np.int64), key_block=np.empty(nu, np.int32), query_chunk=np.empty(nu, np.int32))
    _check(lib.oracle_plan_pairs(_p(cu), ctypes.c_int(n), ctypes.c_int(n_heads), ctypes.c_int(tile), ctypes.c_int(chunk),
                                 ctypes.c_int(n_workers), _p(res["weight"]), _p(res["order"]), _p(res["cta_of_tile"]),
                                 _p(res["cta_offsets"]), _p(res["cta_tiles"]), _p(res["loads"]), _p(res["key_block"]),
                                 _p(res["query_chunk"])), "oracle_plan_pairs")
    res["n_blocks"] = nu
    return res


def vrsp_work(sample_offsets, seq_first_sample):
    """F_i = sum of squared raw-sample lengths of packed sequence i (Eq. 4)."""
    so = _arr(sample_offsets, np.int32)
    fs = _arr(seq_first_sample, np.int32)
    D = len(fs) - 1
    out = np.empty(D, np.int64)
    _check(_load().oracle_vrsp_work(_p(so), _p(fs), ctypes.c_int(D), _p(out)), "oracle_vrsp_work")
    return out


def vrsp_place(work, pool_size):
    """Algorithm 1 -> dict(order, pool_of_seq, pool_load)."""
    w = _arr(work, np.int64)
    D = len(w)
    res = dict(order=np.empty(D, np.int32), pool_of_seq=np.empty(D, np.int32),
               pool_load=np.empty(max(D // pool_size, 1), np.int64))
    _check(_load().oracle_vrsp_place(_p(w), ctypes.c_int(D), ctypes.c_int(pool_size), _p(res["order"]),
                                     _p(res["pool_of_seq"]), _p(res["pool_load"])), "oracle_vrsp_place")
    return res


def tap_place(f, q_home, v_qo, kv_off, kv_grp, v_g, resident, n_workers, tau_num=3, tau_den=100):
    """Algorithm 2 on explicit tile / KV-group tables -> dict(sigma, loads, C, comm_total)."""
    f = _arr(f, np.int64); q_home = _arr(q_home, np.int32); v_qo = _arr(v_qo, np.int64)
    kv_off = _arr(kv_off, np.int32); kv_grp = _arr(kv_grp if len(kv_grp) else [0], np.int32)
    v_g = _arr(v_g if len(v_g) else [0], np.int64); resident = _arr(resident if len(resident) else [-1], np.int32)
    NT, NG, W = len(f), len(v_g), n_workers
    res = dict(sigma=np.empty(NT, np.int32), loads=np.empty(W, np.int64), C=np.empty((W, NG), np.uint8))
    total = ctypes.c_int64(0)
    _check(_load().oracle_tap_place(ctypes.c_int64(NT), ctypes.c_int(W), ctypes.c_int64(NG), _p(f), _p(q_home), _p(v_qo),
                                    _p(kv_off), _p(kv_grp), _p(v_g), _p(resident), ctypes.c_int(tau_num),
                                    ctypes.c_int(tau_den), _p(res["sigma"]), _p(res["loads"]), _p(res["C"]),
                                    ctypes.byref(total)), "oracle_tap_place")
    res["comm_total"] = int(total.value)
    return res


def tap_layout(cu, seq_off, cp, block, n_shards, hq, hkv, d):
    """Tile and KV-group tables of a pool for Algorithm 2 (see oracle_tap_layout)."""
    cu = _arr(cu, np.int32); so = _arr(seq_off, np.int32)
    n, P = len(cu) - 1, len(so) - 1
    lib = _load()
    lib.oracle_tap_num_tiles.restype = ctypes.c_int64
    NT = int(lib.oracle_tap_num_tiles(_p(so), ctypes.c_int(P), ctypes.c_int(block), ctypes.c_int(n_shards)))
    res = dict(f=np.empty(NT, np.int64), q_home=np.empty(NT, np.int32), v_qo=np.empty(NT, np.int64),
               kv_off=np.empty(NT + 1, np.int32), kv_grp=np.empty(NT + n * n_shards + 1, np.int32),
               v_g=np.empty(n * n_shards, np.int64), resident=np.empty(n * n_shards, np.int32))
    _check(lib.oracle_tap_layout(_p(cu), ctypes.c_int(n), _p(so), ctypes.c_int(P), ctypes.c_int(cp), ctypes.c_int(block),
                                 ctypes.c_int(n_shards), ctypes.c_int(hq), ctypes.c_int(hkv), ctypes.c_int(d),
                                 _p(res["f"]), _p(res["q_home"]), _p(res["v_qo"]), _p(res["kv_off"]), _p(res["kv_grp"]),
                                 _p(res["v_g"]), _p(res["resident"])), "oracle_tap_layout")
    res["kv_grp"] = res["kv_grp"][:res["kv_off"][-1]].copy()
    res["n_workers"] = P * cp
    return res


def tap_exchange(cu, seq_off, cp, n_shards, hkv, d, sigma, q_home, v_qo, C, resident):
    """Forward and backward send-byte matrices [src, dst] implied by an assignment."""
    cu = _arr(cu, np.int32); so = _arr(seq_off, np.int32)
    n, P = len(cu) - 1, len(so) - 1
    W = P * cp
    sigma = _arr(sigma, np.int32); q_home = _arr(q_home, np.int32); v_qo = _arr(v_qo, np.int64)
    C = np.ascontiguousarray(C, dtype=np.uint8); resident = _arr(resident, np.int32)
    fwd = np.empty((W, W), np.int64); bwd = np.empty((W, W), np.int64)
    _check(_load().oracle_tap_exchange(_p(cu), ctypes.c_int(n), _p(so), ctypes.c_int(P), ctypes.c_int(cp),
                                       ctypes.c_int(n_shards), ctypes.c_int(hkv), ctypes.c_int(d),
                                       ctypes.c_int64(len(sigma)), _p(sigma), _p(q_home), _p(v_qo), _p(C), _p(resident),
                                       _p(fwd), _p(bwd)), "oracle_tap_exchange")
    return fwd, bwd
