"""ctypes front end of the plain-C float64 oracle.  TEST INFRASTRUCTURE, NOT PRODUCT CODE.

Marshals numpy arrays into ``swaa_oracle.c`` and nothing else: every number the
oracle returns is computed by the C file's plain loops.  Inputs are float32 (or
anything convertible) arrays holding the bf16 input values exactly.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "swaa_oracle.c")
_SO = os.path.join(_HERE, "libswaa_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP over rows) if it is missing or stale."""
    with _lock:
        stale = (not os.path.exists(_SO)) or os.path.getmtime(_SO) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _SO + f".tmp{os.getpid()}"
            subprocess.check_call(
                ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-Wall", "-o", tmp, _SRC, "-lm"]
            )
            os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, i32, dbl, vp = ctypes.c_int64, ctypes.c_int32, ctypes.c_double, ctypes.c_void_p
        lib.swaa_oracle_visible.argtypes = [i64, i64, i64, i64, ctypes.c_int]
        lib.swaa_oracle_visible.restype = ctypes.c_int
        lib.swaa_oracle_count_pairs.argtypes = [i64, i64, i64, ctypes.c_int]
        lib.swaa_oracle_count_pairs.restype = i64
        lib.swaa_oracle_prefill.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i64, i64, ctypes.c_int, dbl, i64,
                                            vp, vp, vp, vp, vp, vp]
        lib.swaa_oracle_prefill.restype = ctypes.c_int
        lib.swaa_oracle_prefill_chunked.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i64, i64, ctypes.c_int, vp,
                                                    dbl, i64, vp, vp, vp, vp, vp, vp]
        lib.swaa_oracle_prefill_chunked.restype = ctypes.c_int
        lib.swaa_oracle_prefill_backward.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i64, i64, ctypes.c_int,
                                                     dbl, vp, vp, vp]
        lib.swaa_oracle_prefill_backward.restype = ctypes.c_int
        lib.swaa_oracle_prefill_backward_rows.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i64, i64,
                                                          ctypes.c_int, dbl, i64, vp, vp, vp, i64, vp, vp, vp, vp]
        lib.swaa_oracle_prefill_backward_rows.restype = ctypes.c_int
        lib.swaa_oracle_decode.argtypes = [vp, vp, vp, vp, i32, i64, i32, i32, i32, i64, i64, ctypes.c_int, dbl,
                                           vp, vp, vp, vp]
        lib.swaa_oracle_decode.restype = ctypes.c_int
        lib.swaa_oracle_layer_is_full.argtypes = [ctypes.c_int] * 5
        lib.swaa_oracle_layer_is_full.restype = ctypes.c_int
        lib.swaa_oracle_layer_is_full_mask.argtypes = [ctypes.c_int, vp, ctypes.c_int, ctypes.c_int]
        lib.swaa_oracle_layer_is_full_mask.restype = ctypes.c_int
        lib.swaa_oracle_select_fa_layers.argtypes = [vp, ctypes.c_int, ctypes.c_int, ctypes.c_int, vp]
        lib.swaa_oracle_select_fa_layers.restype = ctypes.c_int
        lib.swaa_oracle_decode_partial.argtypes = [vp, vp, vp, vp, i32, i64, i64, i32, i32, i32, i64, i64, ctypes.c_int,
                                                   dbl, vp, vp]
        lib.swaa_oracle_decode_partial.restype = ctypes.c_int
        lib.swaa_oracle_decode_combine.argtypes = [vp, ctypes.c_int, i64, ctypes.c_int, vp]
        lib.swaa_oracle_decode_combine.restype = ctypes.c_int
        lib.swaa_oracle_prefill_cp.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i32, i64, i32, i32, i32, i64, i64,
                                               ctypes.c_int, dbl, i64, vp, vp, vp, vp, vp]
        lib.swaa_oracle_prefill_cp.restype = ctypes.c_int
        lib.swaa_oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def visible(i: int, j: int, W: int, S: int, is_full: bool) -> bool:
    return bool(_load().swaa_oracle_visible(i, j, W, S, int(bool(is_full))))


def count_pairs(L: int, W: int, S: int, is_full: bool) -> int:
    return int(_load().swaa_oracle_count_pairs(L, W, S, int(bool(is_full))))


def num_threads() -> int:
    return int(_load().swaa_oracle_num_threads())


def layer_is_full(layer: int, fa_start: int, fa_step: int, fa_decode: bool, phase: int) -> bool:
    return bool(_load().swaa_oracle_layer_is_full(layer, fa_start, fa_step, int(bool(fa_decode)), phase))


def prefill(q, k, v, cu_seqlens, window: int, n_sink: int, is_full: bool, scale: float | None = None, rows=None):
    """Packed varlen prefill.  q [T,Hq,D]; k, v [T,Hkv,D]; cu_seqlens [B+1].

    rows: optional (row_t, row_h) integer arrays selecting (packed token, q-head)
    rows; default all rows in token-major order.  Returns a dict with
    out [n_rows, D] (or [T,Hq,D] for all rows), lse, psum, nvis.
    """
    q, k, v = _f32(q), _f32(k), _f32(v)
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    assert k.shape == (T, Hkv, D) and v.shape == (T, Hkv, D)
    cu = np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int32))
    B = cu.shape[0] - 1
    assert cu[0] == 0 and cu[-1] == T
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    if rows is None:
        n_rows, rt, rh = T * Hq, None, None
    else:
        rt = np.ascontiguousarray(np.asarray(rows[0], dtype=np.int64))
        rh = np.ascontiguousarray(np.asarray(rows[1], dtype=np.int32))
        n_rows = rt.shape[0]
        assert rh.shape[0] == n_rows
    out = np.empty((n_rows, D), dtype=np.float64)
    lse = np.empty(n_rows, dtype=np.float64)
    psum = np.empty(n_rows, dtype=np.float64)
    nvis = np.empty(n_rows, dtype=np.int64)
    rc = _load().swaa_oracle_prefill(_ptr(q), _ptr(k), _ptr(v), _ptr(cu), B, Hq, Hkv, D, int(window), int(n_sink),
                                     int(bool(is_full)), float(scale), n_rows, _ptr(rt), _ptr(rh), _ptr(out),
                                     _ptr(lse), _ptr(psum), _ptr(nvis))
    if rc != 0:
        raise ValueError("swaa_oracle_prefill: inconsistent arguments")
    if rows is None:
        return {"out": out.reshape(T, Hq, D), "lse": lse.reshape(T, Hq), "psum": psum.reshape(T, Hq),
                "nvis": nvis.reshape(T, Hq)}
    return {"out": out, "lse": lse, "psum": psum, "nvis": nvis}


def prefill_chunked(q, k, v, cu_seqlens_q, cu_seqlens_k, window: int, n_sink: int, is_full: bool,
                    scale: float | None = None, rows=None, is_full_seq=None):
    """Chunked prefill: queries are the last len_q tokens of each sequence's len_k-token context.

    q [Tq,Hq,D] packed by cu_seqlens_q; k, v [Tk,Hkv,D] packed by cu_seqlens_k.  rows as in prefill()
    (row_t indexes packed query tokens).  is_full_seq (optional, [B]): a mask policy per sequence, replacing
    is_full.  Returns a dict with out, lse, psum, nvis.
    """
    q, k, v = _f32(q), _f32(k), _f32(v)
    Tq, Hq, D = q.shape
    Tk, Hkv, _ = k.shape
    assert k.shape == (Tk, Hkv, D) and v.shape == (Tk, Hkv, D)
    cq = np.ascontiguousarray(np.asarray(cu_seqlens_q, dtype=np.int32))
    ck = np.ascontiguousarray(np.asarray(cu_seqlens_k, dtype=np.int32))
    B = cq.shape[0] - 1
    assert ck.shape[0] == B + 1 and cq[0] == 0 and ck[0] == 0 and cq[-1] == Tq and ck[-1] == Tk
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    if rows is None:
        n_rows, rt, rh = Tq * Hq, None, None
    else:
        rt = np.ascontiguousarray(np.asarray(rows[0], dtype=np.int64))
        rh = np.ascontiguousarray(np.asarray(rows[1], dtype=np.int32))
        n_rows = rt.shape[0]
        assert rh.shape[0] == n_rows
    out = np.empty((n_rows, D), dtype=np.float64)
    lse = np.empty(n_rows, dtype=np.float64)
    psum = np.empty(n_rows, dtype=np.float64)
    nvis = np.empty(n_rows, dtype=np.int64)
    fs = None if is_full_seq is None else np.ascontiguousarray(np.asarray(is_full_seq, dtype=np.uint8))
    assert fs is None or fs.shape == (B,)
    rc = _load().swaa_oracle_prefill_chunked(_ptr(q), _ptr(k), _ptr(v), _ptr(cq), _ptr(ck), B, Hq, Hkv, D, int(window),
                                             int(n_sink), int(bool(is_full)), _ptr(fs), float(scale), n_rows, _ptr(rt), _ptr(rh),
                                             _ptr(out), _ptr(lse), _ptr(psum), _ptr(nvis))
    if rc != 0:
        raise ValueError("swaa_oracle_prefill_chunked: inconsistent arguments")
    if rows is None:
        return {"out": out.reshape(Tq, Hq, D), "lse": lse.reshape(Tq, Hq), "psum": psum.reshape(Tq, Hq),
                "nvis": nvis.reshape(Tq, Hq)}
    return {"out": out, "lse": lse, "psum": psum, "nvis": nvis}


def decode(q, kcache, vcache, seqlens, window: int, n_sink: int, is_full: bool, scale: float | None = None):
    """Decode.  q [B,Hq,D]; caches [B,Lmax,Hkv,D]; seqlens [B] (valid entries incl. the current token)."""
    q, kcache, vcache = _f32(q), _f32(kcache), _f32(vcache)
    B, Hq, D = q.shape
    _, Lmax, Hkv, _ = kcache.shape
    assert kcache.shape == (B, Lmax, Hkv, D) and vcache.shape == kcache.shape
    sl = np.ascontiguousarray(np.asarray(seqlens, dtype=np.int32))
    assert sl.shape == (B,)
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    out = np.empty((B, Hq, D), dtype=np.float64)
    lse = np.empty((B, Hq), dtype=np.float64)
    psum = np.empty((B, Hq), dtype=np.float64)
    nvis = np.empty((B, Hq), dtype=np.int64)
    rc = _load().swaa_oracle_decode(_ptr(q), _ptr(kcache), _ptr(vcache), _ptr(sl), B, Lmax, Hq, Hkv, D,
                                    int(window), int(n_sink), int(bool(is_full)), float(scale), _ptr(out),
                                    _ptr(lse), _ptr(psum), _ptr(nvis))
    if rc != 0:
        raise ValueError("swaa_oracle_decode: inconsistent arguments")
    return {"out": out, "lse": lse, "psum": psum, "nvis": nvis}


def decode_partial(q, kshard, vshard, seqlens, pos0: int, window: int, n_sink: int, is_full: bool,
                   scale: float | None = None):
    """Partial decode result of one shard of a cache cut along the context.  kshard, vshard [B,Lshard,Hkv,D] hold
    positions pos0 .. pos0+Lshard-1 of every sequence; seqlens are the total lengths.  Returns part [B,Hq,D+2]
    float64 = (max score, sum of exp, unnormalised output) and nvis [B,Hq]."""
    q, kshard, vshard = _f32(q), _f32(kshard), _f32(vshard)
    B, Hq, D = q.shape
    _, Lshard, Hkv, _ = kshard.shape
    assert kshard.shape == (B, Lshard, Hkv, D) and vshard.shape == kshard.shape
    sl = np.ascontiguousarray(np.asarray(seqlens, dtype=np.int32))
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    part = np.empty((B, Hq, D + 2), dtype=np.float64)
    nvis = np.empty((B, Hq), dtype=np.int64)
    rc = _load().swaa_oracle_decode_partial(_ptr(q), _ptr(kshard), _ptr(vshard), _ptr(sl), B, Lshard, int(pos0), Hq, Hkv,
                                            D, int(window), int(n_sink), int(bool(is_full)), float(scale), _ptr(part),
                                            _ptr(nvis))
    if rc != 0:
        raise ValueError("swaa_oracle_decode_partial: inconsistent arguments")
    return {"part": part, "nvis": nvis}


def decode_combine(parts):
    """Log-sum-exp combine of partial decode results.  parts [P,B,Hq,D+2] float64 -> out [B,Hq,D] float64."""
    parts = np.ascontiguousarray(np.asarray(parts, dtype=np.float64))
    P, B, Hq, D2 = parts.shape
    out = np.empty((B, Hq, D2 - 2), dtype=np.float64)
    rc = _load().swaa_oracle_decode_combine(_ptr(parts), P, B * Hq, D2 - 2, _ptr(out))
    if rc != 0:
        raise ValueError("swaa_oracle_decode_combine: inconsistent arguments")
    return out


def prefill_cp(q, k_local, v_local, sink_k, sink_v, cu_seqlens_q, cu_seqlens_k, key_pos0, window: int, n_sink: int,
               is_full: bool, scale: float | None = None, rows=None):
    """Context-parallel prefill of one participant (see swaa_oracle.c): local keys of sequence b start at position
    key_pos0[b]; the queries are the last len_q local positions; sink_k, sink_v [B,sink_rows,Hkv,D] hold positions
    0..sink_rows-1.  Raises ValueError when a visible key is available from neither.  Returns out, lse, nvis."""
    q, k_local, v_local, sink_k, sink_v = _f32(q), _f32(k_local), _f32(v_local), _f32(sink_k), _f32(sink_v)
    Tq, Hq, D = q.shape
    Tk, Hkv, _ = k_local.shape
    cq = np.ascontiguousarray(np.asarray(cu_seqlens_q, dtype=np.int32))
    ck = np.ascontiguousarray(np.asarray(cu_seqlens_k, dtype=np.int32))
    p0 = np.ascontiguousarray(np.asarray(key_pos0, dtype=np.int64))
    B = cq.shape[0] - 1
    assert ck.shape[0] == B + 1 and p0.shape == (B,) and cq[-1] == Tq and ck[-1] == Tk
    sink_rows = sink_k.shape[1]
    assert sink_k.shape == (B, sink_rows, Hkv, D) and sink_v.shape == sink_k.shape
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    if rows is None:
        n_rows, rt, rh = Tq * Hq, None, None
    else:
        rt = np.ascontiguousarray(np.asarray(rows[0], dtype=np.int64))
        rh = np.ascontiguousarray(np.asarray(rows[1], dtype=np.int32))
        n_rows = rt.shape[0]
    out = np.empty((n_rows, D), dtype=np.float64)
    lse = np.empty(n_rows, dtype=np.float64)
    nvis = np.empty(n_rows, dtype=np.int64)
    rc = _load().swaa_oracle_prefill_cp(_ptr(q), _ptr(k_local), _ptr(v_local), _ptr(sink_k), _ptr(sink_v), _ptr(cq),
                                        _ptr(ck), _ptr(p0), B, sink_rows, Hq, Hkv, D, int(window), int(n_sink),
                                        int(bool(is_full)), float(scale), n_rows, _ptr(rt), _ptr(rh), _ptr(out),
                                        _ptr(lse), _ptr(nvis))
    if rc == -2:
        raise ValueError("swaa_oracle_prefill_cp: a visible key is in neither the local keys nor the sink rows")
    if rc != 0:
        raise ValueError("swaa_oracle_prefill_cp: inconsistent arguments")
    if rows is None:
        return {"out": out.reshape(Tq, Hq, D), "lse": lse.reshape(Tq, Hq), "nvis": nvis.reshape(Tq, Hq)}
    return {"out": out, "lse": lse, "nvis": nvis}


def layer_is_full_mask(layer: int, fa_mask, fa_decode: bool, phase: int) -> bool:
    m = np.ascontiguousarray(np.asarray(fa_mask, dtype=np.uint8))
    assert 0 <= layer < m.shape[0]
    return bool(_load().swaa_oracle_layer_is_full_mask(int(layer), _ptr(m), int(bool(fa_decode)), int(phase)))


def select_fa_layers(ratio, n_lazy: int, fa_on_lazy: bool):
    """FA-layer set from per-layer lazy ratios (see swaa_oracle.c).  Returns a uint8 array [n_layers]."""
    r = np.ascontiguousarray(np.asarray(ratio, dtype=np.float64))
    out = np.zeros(r.shape[0], dtype=np.uint8)
    rc = _load().swaa_oracle_select_fa_layers(_ptr(r), r.shape[0], int(n_lazy), int(bool(fa_on_lazy)), _ptr(out))
    if rc != 0:
        raise ValueError("swaa_oracle_select_fa_layers: inconsistent arguments")
    return out


def decode_paged(q, kpages, vpages, block_table, seqlens, window: int, n_sink: int, is_full: bool,
                 scale: float | None = None):
    """Decode against a paged cache, by definition: entry j of sequence b is row j % page_size of page
    block_table[b][j // page_size]; the entries are gathered into a dense cache (pure indexing) and handed
    to the dense decode.  kpages, vpages [num_pages, page_size, Hkv, D]; block_table [B, max_blocks]."""
    kpages, vpages = _f32(kpages), _f32(vpages)
    bt = np.asarray(block_table, dtype=np.int64)
    sl = np.asarray(seqlens, dtype=np.int64)
    B, page_size = bt.shape[0], kpages.shape[1]
    Lmax = int(sl.max())
    kd = np.zeros((B, Lmax) + kpages.shape[2:], dtype=np.float32)
    vd = np.zeros_like(kd)
    for b in range(B):
        j = np.arange(int(sl[b]))
        kd[b, j] = kpages[bt[b, j // page_size], j % page_size]
        vd[b, j] = vpages[bt[b, j // page_size], j % page_size]
    return decode(q, kd, vd, sl, window, n_sink, is_full, scale)


def lazy_ratio(q, k, v_unused, cu_seqlens_q, cu_seqlens_k, recent: int, n_sink: int, scale: float | None = None):
    """Lazy ratio per query head, written out from its definition (App. "Results of LightTransfer"): for every
    given query (the last len_q tokens of each sequence) the full causal softmax over all keys j <= i, then
    the share of it that falls on the last `recent` keys ending at the query or on the first n_sink keys;
    mean over the queries.  Plain float64 numpy loops; v is not needed."""
    q, k = np.asarray(q, dtype=np.float64), np.asarray(k, dtype=np.float64)
    Tq, Hq, D = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    cq, ck = np.asarray(cu_seqlens_q, dtype=np.int64), np.asarray(cu_seqlens_k, dtype=np.int64)
    total = np.zeros(Hq)
    for b in range(cq.shape[0] - 1):
        lq, lk = int(cq[b + 1] - cq[b]), int(ck[b + 1] - ck[b])
        for t in range(lq):
            i = lk - lq + t
            keep = np.array([(j > i - recent) or (j < n_sink) for j in range(i + 1)])
            for h in range(Hq):
                s = (k[ck[b]:ck[b] + i + 1, h // G] @ q[cq[b] + t, h]) * scale
                p = np.exp(s - s.max())
                p /= p.sum()
                total[h] += p[keep].sum()
    return total / Tq


def prefill_paged(q, kpages, vpages, cu_seqlens_q, seqlens_k, block_table, window: int, n_sink: int, is_full: bool,
                  scale: float | None = None, rows=None):
    """Chunked prefill against a paged cache, by definition: the keys and values of each sequence are gathered
    from their pages (pure indexing) into the packed layout and handed to prefill_chunked."""
    kpages, vpages = _f32(kpages), _f32(vpages)
    bt = np.asarray(block_table, dtype=np.int64)
    lk = np.asarray(seqlens_k, dtype=np.int64)
    page_size = kpages.shape[1]
    ks, vs = [], []
    for b in range(bt.shape[0]):
        j = np.arange(int(lk[b]))
        ks.append(kpages[bt[b, j // page_size], j % page_size])
        vs.append(vpages[bt[b, j // page_size], j % page_size])
    cu_k = np.concatenate([[0], np.cumsum(lk)])
    return prefill_chunked(q, np.concatenate(ks), np.concatenate(vs), cu_seqlens_q, cu_k, window, n_sink, is_full, scale,
                           rows)


def prefill_backward_c(q, k, v, dout, cu_seqlens, window: int, n_sink: int, is_full: bool, scale: float | None = None,
                       out_given=None):
    """The same gradients as prefill_backward from the plain-C loops of swaa_oracle.c (fast enough for the sizes of
    the GPU parity tests).  Returns dq [T,Hq,D], dk, dv [T,Hkv,D] float64.

    out_given (optional, [T,Hq,D]): take the row term sum_j p_ij dp_ij as dout_i . out_given_i, i.e. the gradient as
    a function of a stored forward output (see swaa_oracle.c); None: the exact gradient."""
    q, k, v, dout = _f32(q), _f32(k), _f32(v), _f32(dout)
    og = None if out_given is None else _f32(out_given)
    assert og is None or og.shape == q.shape
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    cu = np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int32))
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    dq = np.empty((T, Hq, D), dtype=np.float64)
    dk = np.empty((T, Hkv, D), dtype=np.float64)
    dv = np.empty((T, Hkv, D), dtype=np.float64)
    rc = _load().swaa_oracle_prefill_backward(_ptr(q), _ptr(k), _ptr(v), _ptr(dout), _ptr(og), _ptr(cu), cu.shape[0] - 1, Hq, Hkv, D,
                                              int(window), int(n_sink), int(bool(is_full)), float(scale), _ptr(dq),
                                              _ptr(dk), _ptr(dv))
    if rc != 0:
        raise ValueError("swaa_oracle_prefill_backward: inconsistent arguments")
    return {"dq": dq, "dk": dk, "dv": dv}


def prefill_backward_rows(q, k, v, dout, cu_seqlens, window: int, n_sink: int, is_full: bool, q_rows, kv_rows,
                          scale: float | None = None, out_given=None):
    """Gradients for chosen rows and keys only (plain-C loops, same formulas as prefill_backward_c): dq for the
    (packed token, query head) pairs q_rows = (t, h) and dk, dv for the (packed token, kv head) pairs kv_rows =
    (t, hk).  out_given as in prefill_backward_c.  Returns dq [n_q, D], dk, dv [n_k, D] float64."""
    q, k, v, dout = _f32(q), _f32(k), _f32(v), _f32(dout)
    og = None if out_given is None else _f32(out_given)
    assert og is None or og.shape == q.shape
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    cu = np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int32))
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    qt = np.ascontiguousarray(np.asarray(q_rows[0], dtype=np.int64))
    qh = np.ascontiguousarray(np.asarray(q_rows[1], dtype=np.int32))
    kt = np.ascontiguousarray(np.asarray(kv_rows[0], dtype=np.int64))
    kh = np.ascontiguousarray(np.asarray(kv_rows[1], dtype=np.int32))
    assert qt.shape == qh.shape and kt.shape == kh.shape
    dq = np.empty((qt.shape[0], D), dtype=np.float64)
    dk = np.empty((kt.shape[0], D), dtype=np.float64)
    dv = np.empty((kt.shape[0], D), dtype=np.float64)
    rc = _load().swaa_oracle_prefill_backward_rows(_ptr(q), _ptr(k), _ptr(v), _ptr(dout), _ptr(og), _ptr(cu), cu.shape[0] - 1, Hq,
                                                   Hkv, D, int(window), int(n_sink), int(bool(is_full)), float(scale),
                                                   qt.shape[0], _ptr(qt), _ptr(qh), _ptr(dq), kt.shape[0], _ptr(kt),
                                                   _ptr(kh), _ptr(dk), _ptr(dv))
    if rc != 0:
        raise ValueError("swaa_oracle_prefill_backward_rows: inconsistent arguments")
    return {"dq": dq, "dk": dk, "dv": dv}


def prefill_backward(q, k, v, dout, cu_seqlens, window: int, n_sink: int, is_full: bool, scale: float | None = None):
    """Gradients of the masked softmax attention with respect to q, k, v for an upstream gradient dout, written
    out row by row from the calculus of out_i = sum_j p_ij v_j, p = softmax over the visible keys of scale*q.k:
        dv_j += p_ij dout_i;  dp_ij = dout_i . v_j;  ds_ij = p_ij (dp_ij - sum_j' p_ij' dp_ij');
        dq_i = scale * sum_j ds_ij k_j;  dk_j += scale * ds_ij q_i      (dk, dv summed over the heads of a group).
    Plain float64 numpy; returns dq [T,Hq,D], dk, dv [T,Hkv,D]."""
    q, k, v, dout = (np.asarray(a, dtype=np.float64) for a in (q, k, v, dout))
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    dq, dk, dv = np.zeros_like(q), np.zeros_like(k), np.zeros_like(v)
    for b in range(cu.shape[0] - 1):
        s0, n = int(cu[b]), int(cu[b + 1] - cu[b])
        for i in range(n):
            keys = np.array([j for j in range(i + 1) if visible(i, j, window, n_sink, is_full)], dtype=np.int64) + s0
            for h in range(Hq):
                hk = h // G
                s = (k[keys, hk] @ q[s0 + i, h]) * scale
                p = np.exp(s - s.max())
                p /= p.sum()
                g = dout[s0 + i, h]
                dv[keys, hk] += np.outer(p, g)
                dp = v[keys, hk] @ g
                ds = p * (dp - (p * dp).sum())
                dq[s0 + i, h] = scale * (ds @ k[keys, hk])
                dk[keys, hk] += scale * np.outer(ds, q[s0 + i, h])
    return {"dq": dq, "dk": dk, "dv": dv}
