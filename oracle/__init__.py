"""Float64 CPU oracle for the Pulsar Attention context-encoding path.

TEST INFRASTRUCTURE ONLY: the checker that the CUDA library is compared with.
Nothing in the product path may import this package; it imports nothing from
the product either.  The arithmetic lives in ``pulsar_oracle.c`` (plain C,
float64, OpenMP over independent query rows); this module compiles it with gcc
on first use and marshals numpy arrays through ctypes.

Each wrapper names the passage of the paper its C function follows:

* :func:`maxidf_select` -- Section 3.1 Eq. 2-3, Algorithm 1 line 6, Eq. 4
* :func:`phase1_attn`   -- Eq. 1 over the assembled input of Eq. 4
* :func:`phase2_attn`   -- Section 3.2 / Appendix H (single global softmax)
* :func:`lse_merge`     -- Appendix H Eq. 12-13, iterated
* :func:`generate_step` -- Algorithm 1 lines 11-16 (append KV(q), attend to context + shard)
* :func:`causal_varlen_attn` -- Eq. 1 over whole assembled inputs (Algorithm 1 line 8)
* :func:`chunk_select`  -- Appendix C: TF-IDF, BM25, type-token and Max-IDF chunk scores
* :func:`assemble_positions`, :func:`rope_apply` -- Appendix E: position ids and rotary embedding
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pulsar_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle into ``oracle/liboracle.so`` (gcc, -O2, OpenMP)."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.check_call(
                ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32, i64, f64, vp = ctypes.c_int32, ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        lib.oracle_maxidf_select.argtypes = [vp, i64, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp]
        lib.oracle_maxidf_select.restype = ctypes.c_int
        lib.oracle_phase1_attn.argtypes = [vp, vp, vp, i64, i32, i32, i32, i32, vp, vp, i32, f64,
                                           vp, i64, vp, vp]
        lib.oracle_phase1_attn.restype = ctypes.c_int
        lib.oracle_phase2_attn.argtypes = [vp, i32, vp, vp, i32, i32, i32, i32, i32, f64,
                                           vp, vp, vp, vp]
        lib.oracle_phase2_attn.restype = ctypes.c_int
        lib.oracle_lse_merge.argtypes = [vp, vp, i32, i64, i32, vp, vp]
        lib.oracle_generate_step.argtypes = [vp, vp, vp, i32, vp, vp, i64, vp, vp, i32, i32, i32, i32, i32, f64, vp, vp]
        lib.oracle_generate_step.restype = ctypes.c_int
        lib.oracle_lse_merge.restype = ctypes.c_int
        lib.oracle_chunk_select.argtypes = [vp, i64, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp]
        lib.oracle_chunk_select.restype = ctypes.c_int
        lib.oracle_assemble_positions.argtypes = [vp, vp, i32, i32, i32, vp]
        lib.oracle_assemble_positions.restype = ctypes.c_int64
        lib.oracle_rope_apply.argtypes = [vp, i64, i32, i32, vp, ctypes.c_double, vp]
        lib.oracle_rope_apply.restype = ctypes.c_int
        _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _bits(x) -> np.ndarray:
    """bf16 payload as a C-contiguous uint16 array (torch.bfloat16 or uint16 ndarray)."""
    if isinstance(x, np.ndarray):
        assert x.dtype == np.uint16
        return np.ascontiguousarray(x)
    import torch  # only to reinterpret a CPU bf16 tensor's bits
    assert x.dtype == torch.bfloat16 and x.device.type == "cpu"
    return np.ascontiguousarray(x.contiguous().view(torch.int16).numpy().view(np.uint16))


def num_threads() -> int:
    """Threads the OpenMP regions use (OMP_NUM_THREADS if set, else all cores)."""
    env = os.environ.get("OMP_NUM_THREADS")
    return int(env) if env else (os.cpu_count() or 1)


def maxidf_select(token_ids, vocab_size, block_size, chunk, k, sink):
    """Max-IDF summary selection.  Returns a dict with ``sel_chunks`` [B,k],
    ``prefix_idx`` [sink+(B-1)*k*chunk], ``prefix_len`` [B], ``df`` [V] (uint32),
    ``idf`` [V] and ``score`` [B, C] (float64), B = ceil(L/block_size) blocks of
    C = ceil(block_size/chunk) chunk slots.  Where a block has fewer than k chunks the
    row of ``sel_chunks`` ends in -1; unused entries of ``prefix_idx`` are -1."""
    ids = np.ascontiguousarray(np.asarray(token_ids, dtype=np.uint32))
    L = ids.shape[0]
    B, C = -(-L // block_size), -(-block_size // chunk)
    sel = np.zeros((B, k), np.int32)
    pidx = np.zeros(sink + max(B - 1, 0) * k * chunk, np.int32)
    plen = np.zeros(B, np.int32)
    df = np.zeros(vocab_size, np.uint32)
    idf = np.zeros(vocab_size, np.float64)
    score = np.zeros((B, C), np.float64)
    rc = _load().oracle_maxidf_select(_ptr(ids), L, vocab_size, block_size, chunk, k, sink,
                                      _ptr(sel), _ptr(pidx), _ptr(plen), _ptr(df), _ptr(idf),
                                      _ptr(score))
    if rc != 0:
        raise ValueError(f"oracle_maxidf_select rejected the shape (rc={rc})")
    return dict(sel_chunks=sel, prefix_idx=pidx, prefix_len=plen, df=df, idf=idf, score=score)


def phase1_attn(Q, K, V, block_size, prefix_idx, prefix_len, scale=0.0, rows=None):
    """Phase-1 prefix-block attention for the query positions ``rows`` (all if
    None).  Q [L,Hq,d], K,V [L,Hkv,d] bf16.  Returns (O [n,Hq,d], LSE [n,Hq]) float64."""
    q, kk, v = _bits(Q), _bits(K), _bits(V)
    L, Hq, d = q.shape
    Hkv = kk.shape[1]
    pidx = np.ascontiguousarray(np.asarray(prefix_idx, dtype=np.int32))
    plen = np.ascontiguousarray(np.asarray(prefix_len, dtype=np.int32))
    r = None if rows is None else np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    n = L if r is None else r.shape[0]
    O = np.zeros((n, Hq, d), np.float64)
    LSE = np.zeros((n, Hq), np.float64)
    rc = _load().oracle_phase1_attn(_ptr(q), _ptr(kk), _ptr(v), L, Hq, Hkv, d, block_size,
                                    _ptr(pidx), _ptr(plen), pidx.shape[0], float(scale),
                                    _ptr(r), n, _ptr(O), _ptr(LSE))
    if rc != 0:
        raise ValueError(f"oracle_phase1_attn rejected its arguments (rc={rc})")
    return O, LSE


def phase2_attn(Qq, K, V, n_blocks, block_size, scale=0.0, partials=False):
    """Phase-2 query attention over all retained KV.  Qq [nq,Hq,d], K,V
    [n_blocks*block_size,Hkv,d] bf16.  Returns (O, LSE) or, with ``partials``,
    (O, LSE, part_O [B,nq,Hq,d], part_LSE [B,nq,Hq]); all float64."""
    q, kk, v = _bits(Qq), _bits(K), _bits(V)
    nq, Hq, d = q.shape
    Hkv = kk.shape[1]
    assert kk.shape[0] == n_blocks * block_size
    O = np.zeros((nq, Hq, d), np.float64)
    LSE = np.zeros((nq, Hq), np.float64)
    pO = np.zeros((n_blocks, nq, Hq, d), np.float64) if partials else None
    pL = np.zeros((n_blocks, nq, Hq), np.float64) if partials else None
    rc = _load().oracle_phase2_attn(_ptr(q), nq, _ptr(kk), _ptr(v), n_blocks, block_size,
                                    Hq, Hkv, d, float(scale), _ptr(O), _ptr(LSE), _ptr(pO), _ptr(pL))
    if rc != 0:
        raise ValueError(f"oracle_phase2_attn rejected its arguments (rc={rc})")
    return (O, LSE, pO, pL) if partials else (O, LSE)


def lse_merge(part_O, part_LSE):
    """Iterated online-softmax merge.  part_O [J,rows,d], part_LSE [J,rows] float64."""
    pO = np.ascontiguousarray(np.asarray(part_O, dtype=np.float64))
    pL = np.ascontiguousarray(np.asarray(part_LSE, dtype=np.float64))
    J, rows, d = pO.shape
    O = np.zeros((rows, d), np.float64)
    LSE = np.zeros(rows, np.float64)
    rc = _load().oracle_lse_merge(_ptr(pO), _ptr(pL), J, rows, d, _ptr(O), _ptr(LSE))
    if rc != 0:
        raise ValueError(f"oracle_lse_merge rejected its arguments (rc={rc})")
    return O, LSE


def generate_step(Qnew, Knew, Vnew, Kctx, Vctx, Kgen_bits, Vgen_bits, gen_len, scale=0.0):
    """One generation step.  Qnew [n,Hq,d], Knew/Vnew [n,Hkv,d], Kctx/Vctx [L,Hkv,d] bf16;
    Kgen_bits/Vgen_bits: uint16 ndarrays [capacity,Hkv,d] holding the shard's bf16 patterns,
    updated in place (rows gen_len .. gen_len+n).  Returns (O [n,Hq,d], LSE [n,Hq]) float64."""
    q, kn, vn, kc, vc = _bits(Qnew), _bits(Knew), _bits(Vnew), _bits(Kctx), _bits(Vctx)
    assert Kgen_bits.dtype == np.uint16 and Kgen_bits.flags.c_contiguous and Vgen_bits.flags.c_contiguous
    n, Hq, d = q.shape
    Hkv = kc.shape[1]
    O = np.zeros((n, Hq, d), np.float64)
    LSE = np.zeros((n, Hq), np.float64)
    rc = _load().oracle_generate_step(_ptr(q), _ptr(kn), _ptr(vn), n, _ptr(kc), _ptr(vc), kc.shape[0],
                                      _ptr(Kgen_bits), _ptr(Vgen_bits), gen_len, Kgen_bits.shape[0], Hq, Hkv, d,
                                      float(scale), _ptr(O), _ptr(LSE))
    if rc != 0:
        raise ValueError(f"oracle_generate_step rejected its arguments (rc={rc})")
    return O, LSE


def causal_varlen_attn(Q, K, V, cu_seqlens, scale=0.0):
    """Causal attention inside each of the sequences packed back to back (Eq. 1 over every
    assembled input of Eq. 4, all rows as queries).  Each sequence is one block without a
    prefix.  Q [T,Hq,d], K,V [T,Hkv,d] bf16.  Returns (O [T,Hq,d], LSE [T,Hq]) float64."""
    q, kk, v = _bits(Q), _bits(K), _bits(V)
    T, Hq, d = q.shape
    O = np.zeros((T, Hq, d), np.float64)
    LSE = np.zeros((T, Hq), np.float64)
    none = np.zeros(0, np.int32)
    for a, b in zip(cu_seqlens[:-1], cu_seqlens[1:]):
        O[a:b], LSE[a:b] = phase1_attn(q[a:b], kk[a:b], v[a:b], b - a, none, np.zeros(1, np.int32), scale)
    return O, LSE


SCORE_MODES = {"max_idf": 0, "tf_idf": 1, "bm25": 2, "type_token": 3}


def chunk_select(token_ids, vocab_size, block_size, chunk, k, sink, mode):
    """Chunk selection under one of the Appendix C heuristics (``mode`` a key of SCORE_MODES or
    its number).  Returns sel_chunks [B,k], prefix_idx, prefix_len and score [B,C] (float64);
    B = ceil(L/block_size), C = ceil(block_size/chunk), padding as in :func:`maxidf_select`."""
    ids = np.ascontiguousarray(np.asarray(token_ids, dtype=np.uint32))
    L = ids.shape[0]
    B, C = -(-L // block_size), -(-block_size // chunk)
    m = SCORE_MODES.get(mode, mode)
    sel = np.zeros((B, k), np.int32)
    pidx = np.zeros(sink + max(B - 1, 0) * k * chunk, np.int32)
    plen = np.zeros(B, np.int32)
    score = np.zeros((B, C), np.float64)
    rc = _load().oracle_chunk_select(_ptr(ids), L, vocab_size, block_size, chunk, k, sink, int(m),
                                     _ptr(sel), _ptr(pidx), _ptr(plen), _ptr(score))
    if rc != 0:
        raise ValueError(f"oracle_chunk_select rejected its arguments (rc={rc})")
    return dict(sel_chunks=sel, prefix_idx=pidx, prefix_len=plen, score=score)


def assemble_positions(prefix_idx, prefix_len, block_size, mode="sparse"):
    """Position ids of the assembled Phase-1 inputs stored back to back (Appendix E); ``mode``
    "sparse" (global positions kept) or "contiguous" (each input renumbered from 0)."""
    pidx = np.ascontiguousarray(np.asarray(prefix_idx, dtype=np.int32))
    plen = np.ascontiguousarray(np.asarray(prefix_len, dtype=np.int32))
    B = plen.shape[0]
    out = np.zeros(int(plen.sum()) + B * block_size, np.int32)
    n = _load().oracle_assemble_positions(_ptr(pidx), _ptr(plen), B, block_size,
                                          {"sparse": 0, "contiguous": 1}[mode], _ptr(out))
    if n != out.shape[0]:
        raise ValueError("oracle_assemble_positions rejected its arguments")
    return out


def rope_apply(X, positions, theta=500000.0):
    """Rotary embedding (rotate-half pairing) of X [rows,H,d] bf16 at the given position ids.
    Returns float64 [rows,H,d]."""
    x = _bits(X)
    rows, H, d = x.shape
    pos = np.ascontiguousarray(np.asarray(positions, dtype=np.int32))
    Y = np.zeros((rows, H, d), np.float64)
    rc = _load().oracle_rope_apply(_ptr(x), rows, H, d, _ptr(pos), float(theta), _ptr(Y))
    if rc != 0:
        raise ValueError(f"oracle_rope_apply rejected its arguments (rc={rc})")
    return Y
