"""CPU oracle package (test infrastructure, not part of the product).

`lib()` loads liboracle.so, built from spec_oracle.c by `build()` (plain gcc, no CUDA).  Only the tests, the
smoke check and the benchmark's CPU-baseline leg may import this package; the CUDA library never does.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "liboracle.so")
_SRC = os.path.join(_HERE, "spec_oracle.c")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-o", _SO, _SRC, "-lm"])
    return _SO


def lib():
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_SO)
        c = ctypes
        f32p, i32p, u32p, f64p = (c.POINTER(c.c_float), c.POINTER(c.c_int32), c.POINTER(c.c_uint32),
                                  c.POINTER(c.c_double))
        L.spec_oracle_philox4x32_10.argtypes = [u32p, u32p, u32p]
        L.spec_oracle_uniform.argtypes = [c.c_uint64, c.c_uint32, c.c_uint32, c.c_uint32, c.c_uint32]
        L.spec_oracle_uniform.restype = c.c_float
        L.spec_oracle_uniforms.argtypes = [c.c_uint64, c.c_uint32, c.c_uint32, c.c_int, c.c_int, f32p]
        L.spec_oracle_softmax.argtypes = [f32p, c.c_int, c.c_int, c.c_double, f32p]
        L.spec_oracle_softmax_row.argtypes = [f32p, c.c_int, c.c_double, f32p, f64p, f64p]
        L.spec_oracle_logprob.argtypes = [f32p, c.c_int, c.c_double, c.c_int]
        L.spec_oracle_logprob.restype = c.c_double
        L.spec_oracle_invcdf_f32.argtypes = [f32p, c.c_int, c.c_float, f64p]
        L.spec_oracle_invcdf_f32.restype = c.c_int
        L.spec_oracle_reject_sample_seq.argtypes = [c.c_int, c.c_int, f32p, f32p, i32p, f32p, i32p, i32p, u32p, f64p]
        L.spec_oracle_reject_sample.argtypes = [c.c_int, c.c_int, c.c_int, f32p, f32p, i32p, c.c_uint64,
                                                c.c_uint32, i32p, i32p, u32p, f64p]
        L.spec_oracle_sample_rows.argtypes = [c.c_int, c.c_int, f32p, f32p, i32p, f64p]
        L.spec_oracle_kv_reserve.argtypes = [c.c_int, c.c_int, c.c_int, c.c_int, i32p, i32p, i32p, i32p]
        L.spec_oracle_kv_reserve.restype = c.c_int
        L.spec_oracle_kv_commit.argtypes = [c.c_int, c.c_int, c.c_int, i32p, i32p, i32p, i32p, i32p]
        L.spec_oracle_kv_replace.argtypes = [c.c_int, i32p, i32p, c.c_int, c.c_int, i32p, i32p, i32p, i32p]
        L.spec_oracle_kv_replace.restype = c.c_int
        L.spec_oracle_e4m3_quantize.argtypes = [c.c_size_t, c.POINTER(c.c_float), c.c_float, c.POINTER(c.c_uint8)]
        L.spec_oracle_e4m3_quantize_rows.argtypes = [c.c_size_t, c.c_size_t, c.POINTER(c.c_float), c.POINTER(c.c_float), c.POINTER(c.c_uint8)]
        L.spec_oracle_e4m3_quantize_rows.restype = None
        L.spec_oracle_e4m3_dequantize.argtypes = [c.c_size_t, c.POINTER(c.c_uint8), c.c_float, c.POINTER(c.c_float)]
        _lib = L
    return _lib


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


# ---- thin numpy-facing wrappers (marshalling only) -------------------------------------------------------

def philox4x32_10(ctr, key):
    c = np.ascontiguousarray(ctr, np.uint32)
    k = np.ascontiguousarray(key, np.uint32)
    out = np.zeros(4, np.uint32)
    lib().spec_oracle_philox4x32_10(_p(c, ctypes.c_uint32), _p(k, ctypes.c_uint32), _p(out, ctypes.c_uint32))
    return out


def uniform(seed, step, seq, slot, stream):
    return float(lib().spec_oracle_uniform(seed, step, seq, slot, stream))


def uniforms(seed, step, stream, n_seq, n_slots):
    u = np.zeros((n_seq, n_slots), np.float32)
    lib().spec_oracle_uniforms(seed, step, stream, n_seq, n_slots, _p(u, ctypes.c_float))
    return u


def softmax(logits, temperature=1.0):
    lg = _f32(logits)
    V = lg.shape[-1]
    rows = lg.size // V
    out = np.empty_like(lg)
    lib().spec_oracle_softmax(_p(lg, ctypes.c_float), rows, V, float(temperature), _p(out, ctypes.c_float))
    return out


def softmax_stats(logits_row, temperature=1.0):
    lg = _f32(logits_row)
    m, z = ctypes.c_double(), ctypes.c_double()
    lib().spec_oracle_softmax_row(_p(lg, ctypes.c_float), lg.shape[0], float(temperature), None,
                                  ctypes.byref(m), ctypes.byref(z))
    return m.value, z.value


def logprob(logits_row, token, temperature=1.0):
    lg = _f32(logits_row)
    return float(lib().spec_oracle_logprob(_p(lg, ctypes.c_float), lg.shape[0], float(temperature), int(token)))


def invcdf(weights, u):
    w = _f32(weights)
    mg = ctypes.c_double()
    t = lib().spec_oracle_invcdf_f32(_p(w, ctypes.c_float), w.shape[0], float(u), ctypes.byref(mg))
    return int(t), mg.value


def sample_rows(probs, u):
    pr = _f32(probs)
    uu = _f32(u)
    B, V = pr.shape
    tok = np.zeros(B, np.int32)
    mg = np.zeros(B, np.float64)
    lib().spec_oracle_sample_rows(B, V, _p(pr, ctypes.c_float), _p(uu, ctypes.c_float), _p(tok, ctypes.c_int32),
                                  _p(mg, ctypes.c_double))
    return tok, mg


def reject_sample_seq(p, q, draft, u):
    """One sequence: p [k+1][V], q [k][V], draft [k], u [k+1] -> (out_tokens [k+1], n_emitted, flags, margins)."""
    p, q, draft, u = _f32(p), _f32(q), _i32(draft), _f32(u)
    k, V = q.shape[0], p.shape[1]
    assert p.shape[0] == k + 1 and u.shape[0] == k + 1
    out = np.zeros(k + 1, np.int32)
    n = ctypes.c_int32()
    fl = ctypes.c_uint32()
    mg = np.zeros(k + 1, np.float64)
    qq = q if k > 0 else np.zeros((1, V), np.float32)
    dd = draft if k > 0 else np.zeros(1, np.int32)
    lib().spec_oracle_reject_sample_seq(k, V, _p(p, ctypes.c_float), _p(qq, ctypes.c_float), _p(dd, ctypes.c_int32),
                                        _p(u, ctypes.c_float), _p(out, ctypes.c_int32), ctypes.byref(n),
                                        ctypes.byref(fl), _p(mg, ctypes.c_double))
    return out, n.value, fl.value, mg


def reject_sample(p, q, draft, seed, step):
    """Batch: p [B][k+1][V], q [B][k][V], draft [B][k]; uniforms are Philox(seed; step, b, slot, 0)."""
    p, q, draft = _f32(p), _f32(q), _i32(draft)
    B, kp1, V = p.shape
    k = kp1 - 1
    out = np.zeros((B, k + 1), np.int32)
    n = np.zeros(B, np.int32)
    fl = np.zeros(B, np.uint32)
    mg = np.zeros((B, k + 1), np.float64)
    qq = q if k > 0 else np.zeros((1,), np.float32)
    dd = draft if k > 0 else np.zeros((1,), np.int32)
    lib().spec_oracle_reject_sample(B, k, V, _p(p, ctypes.c_float), _p(qq, ctypes.c_float), _p(dd, ctypes.c_int32),
                                    seed, step, _p(out, ctypes.c_int32), _p(n, ctypes.c_int32),
                                    _p(fl, ctypes.c_uint32), _p(mg, ctypes.c_double))
    return out, n, fl, mg


def kv_reserve(k, block_tokens, seq_len, block_table, free_stack, free_top):
    """In place on int32 arrays; free_top is a 1-element int32 array.  Returns 0, or <0 if it cannot be served."""
    B, max_blocks = block_table.shape
    return lib().spec_oracle_kv_reserve(B, k, block_tokens, max_blocks, _p(seq_len, ctypes.c_int32),
                                        _p(block_table, ctypes.c_int32), _p(free_stack, ctypes.c_int32),
                                        _p(free_top, ctypes.c_int32))


def kv_commit(block_tokens, n_emitted, seq_len, block_table, free_stack, free_top):
    B, max_blocks = block_table.shape
    ne = _i32(n_emitted)
    lib().spec_oracle_kv_commit(B, block_tokens, max_blocks, _p(ne, ctypes.c_int32), _p(seq_len, ctypes.c_int32),
                                _p(block_table, ctypes.c_int32), _p(free_stack, ctypes.c_int32),
                                _p(free_top, ctypes.c_int32))


def kv_replace(slots, new_len, block_tokens, seq_len, block_table, free_stack, free_top):
    sl, nl = _i32(slots), _i32(new_len)
    B, max_blocks = block_table.shape
    return lib().spec_oracle_kv_replace(sl.shape[0], _p(sl, ctypes.c_int32), _p(nl, ctypes.c_int32), block_tokens, max_blocks,
                                        _p(seq_len, ctypes.c_int32), _p(block_table, ctypes.c_int32),
                                        _p(free_stack, ctypes.c_int32), _p(free_top, ctypes.c_int32))


def kv_compact(keep, block_tokens, seq_len, block_table, free_stack, free_top):
    """Shrinks the batch to the sequences in the (strictly ascending) slots `keep`: every other slot is retired in slot
    order (kv_replace with a negative length: its blocks go back to the free stack in logical order), then new slot j takes
    old slot keep[j]'s length and table row.  Returns (seq_len, block_table) of the len(keep) remaining sequences; the free
    stack is updated in place.  (Continuous batching, paper Section 5.2: the long tail of a rollout runs on a thin batch.)"""
    keep = [int(k) for k in keep]
    assert all(a < b for a, b in zip(keep, keep[1:])) and all(0 <= k < seq_len.shape[0] for k in keep)
    dropped = [b for b in range(seq_len.shape[0]) if b not in keep]
    if dropped:
        assert kv_replace(dropped, [-1] * len(dropped), block_tokens, seq_len, block_table, free_stack, free_top) == 0
    return seq_len[keep].copy(), block_table[keep].copy()


def e4m3_quantize(x, scale=1.0):
    """e4m3 codes (uint8) of x / scale: round to nearest even, saturating at 448."""
    xf = _f32(x)
    out = np.empty(xf.shape, np.uint8)
    lib().spec_oracle_e4m3_quantize(xf.size, _p(xf, ctypes.c_float), float(scale), _p(out, ctypes.c_uint8))
    return out


def e4m3_quantize_rows(x):
    """Per-row e4m3 codes and scales of a matrix [rows][k]: scale = amax(row) / 448 (1 for a zero row)."""
    xf = _f32(x)
    assert xf.ndim == 2
    codes = np.empty(xf.shape, np.uint8)
    scales = np.empty(xf.shape[0], np.float32)
    lib().spec_oracle_e4m3_quantize_rows(xf.shape[0], xf.shape[1], _p(xf, ctypes.c_float), _p(scales, ctypes.c_float), _p(codes, ctypes.c_uint8))
    return codes, scales


def e4m3_rows_roundtrip(x):
    """x with every row replaced by its 8-bit representation (codes times the row's scale), fp32."""
    codes, scales = e4m3_quantize_rows(x)
    return (e4m3_dequantize(codes, 1.0).reshape(codes.shape) * scales[:, None]).astype(np.float32)


def e4m3_dequantize(codes, scale=1.0):
    cc = np.ascontiguousarray(codes, np.uint8)
    out = np.empty(cc.shape, np.float32)
    lib().spec_oracle_e4m3_dequantize(cc.size, _p(cc, ctypes.c_uint8), float(scale), _p(out, ctypes.c_float))
    return out


def e4m3_roundtrip(x, scale=1.0):
    return e4m3_dequantize(e4m3_quantize(x, scale), scale)
