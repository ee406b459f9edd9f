"""ctypes binding of the Pulsar CUDA library (``include/pulsar.h``).

Argument marshalling only: tensors in, device pointers and sizes through the C
ABI, tensors out.  Every step of the path runs in the library's kernels.  torch
provides device memory and the stream; nothing here computes.  The library is
required: if it is missing the first call raises, there is no fallback.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import _build

_HERE = os.path.dirname(os.path.abspath(__file__))
_lib = None

STATUS_NAMES = {
    0: "PULSAR_OK", 1: "PULSAR_ERR_INVALID_ARG", 2: "PULSAR_ERR_SHAPE", 3: "PULSAR_ERR_ALIGNMENT",
    4: "PULSAR_ERR_WORKSPACE", 5: "PULSAR_ERR_UNSUPPORTED_DEVICE", 6: "PULSAR_ERR_CUDA",
    7: "PULSAR_ERR_TIMEOUT", 8: "PULSAR_ERR_DEVICE_CHECK",
}
DEV_BAD_TOKEN, DEV_BAD_PREFIX, DEV_TIMEOUT, DEV_BAD_LENGTH, DEV_BAD_POSITION = 0x1, 0x2, 0x4, 0x8, 0x10

EXPORTS = (
    "pulsar_status_string", "pulsar_abi_version", "pulsar_launch_count", "pulsar_wait_selftest",
    "pulsar_maxidf_select_workspace_bytes", "pulsar_maxidf_select",
    "pulsar_maxidf_select_noalloc_max_scratch", "pulsar_maxidf_select_noalloc",
    "pulsar_chunk_select_workspace_bytes", "pulsar_chunk_select",
    "pulsar_phase1_workspace_bytes", "pulsar_phase1_attn",
    "pulsar_pack_summary_kv", "pulsar_gather_kv_rows", "pulsar_phase1_attn_sharded", "pulsar_causal_varlen_attn",
    "pulsar_retain_block_kv",
    "pulsar_phase2_choose_splits", "pulsar_phase2_workspace_bytes", "pulsar_phase2_attn",
    "pulsar_phase2_generate_workspace_bytes", "pulsar_phase2_generate_step",
    "pulsar_lse_merge", "pulsar_lse_merge_strided", "pulsar_lse_merge_peers",
    "pulsar_assemble_positions", "pulsar_rope_apply", "pulsar_rope_apply_qk",
)


class PulsarError(RuntimeError):
    def __init__(self, call: str, status: int):
        self.status = status
        super().__init__(f"{call} failed: {STATUS_NAMES.get(status, status)}")


def library_path() -> str:
    """Path of the CUDA library: the in-tree build, or $PULSAR_LIBRARY if set (a custom build)."""
    return os.environ.get("PULSAR_LIBRARY") or _build.LIB


def load_library(build_if_missing: bool = False):
    """Load ``libpulsar.so`` (built in-tree).  Raises if it does not exist."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        if build_if_missing:
            _build.build()
        else:
            raise FileNotFoundError(
                f"{path} is missing: build it with `python -m paper_2607_20457_b200._build` "
                "(the CUDA library is the only implementation; there is no CPU path)")
    lib = ctypes.CDLL(path)
    i32, i64, vp, sz, f32 = ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_float
    lib.pulsar_status_string.argtypes = [i32]
    lib.pulsar_status_string.restype = ctypes.c_char_p
    lib.pulsar_abi_version.argtypes = []
    lib.pulsar_abi_version.restype = i32
    lib.pulsar_launch_count.argtypes = []
    lib.pulsar_launch_count.restype = ctypes.c_uint64
    lib.pulsar_wait_selftest.argtypes = [vp, ctypes.c_uint64, vp, vp]
    lib.pulsar_wait_selftest.restype = i32
    lib.pulsar_maxidf_select_workspace_bytes.argtypes = [i64, i32, i32, i32, i32, i32]
    lib.pulsar_maxidf_select_workspace_bytes.restype = sz
    lib.pulsar_maxidf_select.argtypes = [vp, i64, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, sz, vp, vp]
    lib.pulsar_maxidf_select.restype = i32
    lib.pulsar_maxidf_select_noalloc_max_scratch.argtypes = []
    lib.pulsar_maxidf_select_noalloc_max_scratch.restype = sz
    lib.pulsar_maxidf_select_noalloc.argtypes = [vp, i64, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.pulsar_maxidf_select_noalloc.restype = i32
    lib.pulsar_chunk_select_workspace_bytes.argtypes = [i64, i32, i32, i32, i32, i32, i32]
    lib.pulsar_chunk_select_workspace_bytes.restype = sz
    lib.pulsar_chunk_select.argtypes = [vp, i64, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, sz, vp, vp]
    lib.pulsar_chunk_select.restype = i32
    lib.pulsar_phase1_workspace_bytes.argtypes = [i64, i32, i32, i32, i32, i32]
    lib.pulsar_phase1_workspace_bytes.restype = sz
    lib.pulsar_phase1_attn.argtypes = [vp, vp, vp, i64, i32, i32, i32, i32, vp, vp, i32, f32,
                                       vp, vp, vp, vp, vp, sz, vp, vp]
    lib.pulsar_phase1_attn.restype = i32
    lib.pulsar_pack_summary_kv.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp, i32, i32, i32, i32, vp, vp, vp, vp]
    lib.pulsar_pack_summary_kv.restype = i32
    lib.pulsar_gather_kv_rows.argtypes = [vp, vp, i64, i32, i32, vp, i32, vp, vp, vp, vp]
    lib.pulsar_gather_kv_rows.restype = i32
    lib.pulsar_phase1_attn_sharded.argtypes = [vp, vp, vp, i64, i32, i32, i32, i32, vp, vp, i32, vp, f32, vp, vp,
                                               vp, sz, vp, vp]
    lib.pulsar_phase1_attn_sharded.restype = i32
    lib.pulsar_lse_merge_strided.argtypes = [vp, vp, i32, i64, i64, i64, i32, vp, i32, vp, vp]
    lib.pulsar_lse_merge_strided.restype = i32
    lib.pulsar_causal_varlen_attn.argtypes = [vp, vp, vp, i64, vp, i32, i32, i32, i32, f32, vp, vp, vp, sz, vp, vp]
    lib.pulsar_causal_varlen_attn.restype = i32
    lib.pulsar_phase2_choose_splits.argtypes = [i32, i32, i32, i32, i32, i32]
    lib.pulsar_phase2_choose_splits.restype = i32
    lib.pulsar_phase2_workspace_bytes.argtypes = [i32, i32, i32, i32, i32, i32, i32]
    lib.pulsar_phase2_workspace_bytes.restype = sz
    lib.pulsar_phase2_attn.argtypes = [vp, i32, vp, vp, i32, i32, i32, i32, i32, f32, i32,
                                       vp, vp, vp, vp, vp, sz, vp, vp]
    lib.pulsar_phase2_attn.restype = i32
    lib.pulsar_phase2_generate_workspace_bytes.argtypes = [i32, i32, i32, i32, i32, i32, i32]
    lib.pulsar_phase2_generate_workspace_bytes.restype = sz
    lib.pulsar_phase2_generate_step.argtypes = [vp, vp, vp, i32, vp, vp, i32, i32, vp, vp, i32, i32, i32, i32, i32,
                                                f32, i32, vp, vp, vp, sz, vp, vp]
    lib.pulsar_phase2_generate_step.restype = i32
    lib.pulsar_lse_merge.argtypes = [vp, vp, i32, i64, i32, vp, vp, vp]
    lib.pulsar_lse_merge.restype = i32
    lib.pulsar_lse_merge_peers.argtypes = [vp, i32, i64, i64, i64, i32, vp, i32, vp, vp]
    lib.pulsar_lse_merge_peers.restype = i32
    lib.pulsar_retain_block_kv.argtypes = [vp, vp, i64, vp, i32, i32, i32, i32, vp, vp, vp]
    lib.pulsar_retain_block_kv.restype = i32
    lib.pulsar_assemble_positions.argtypes = [vp, vp, i32, i32, i32, i32, vp, i64, vp, vp]
    lib.pulsar_assemble_positions.restype = i32
    lib.pulsar_rope_apply.argtypes = [vp, vp, i64, i32, i32, vp, ctypes.c_double, vp, vp]
    lib.pulsar_rope_apply.restype = i32
    lib.pulsar_rope_apply_qk.argtypes = [vp, vp, i32, vp, vp, i32, i64, i32, vp, ctypes.c_double, vp, vp]
    lib.pulsar_rope_apply_qk.restype = i32
    _lib = lib
    return lib


def _p(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(call: str, rc: int):
    if rc != 0:
        raise PulsarError(call, rc)


def _need(t: torch.Tensor, dtype, name: str):
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of {dtype}, got {t.dtype} on {t.device}")


def _workspace(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def launch_count() -> int:
    """Kernels launched by the library in this process so far."""
    return int(load_library().pulsar_launch_count())


def wait_selftest(limit_ns: int, status: torch.Tensor, result: torch.Tensor):
    """Run the bounded-wait self-test kernel (see pulsar_wait_selftest)."""
    _check("pulsar_wait_selftest", load_library().pulsar_wait_selftest(_p(status), int(limit_ns), _p(result), _stream()))


def new_status(device) -> torch.Tensor:
    """A zeroed device status word for the kernels' data-dependent checks."""
    return torch.zeros(1, dtype=torch.int32, device=device)


def maxidf_select_workspace_bytes(L, vocab_size, block_size, chunk, k, sink) -> int:
    return load_library().pulsar_maxidf_select_workspace_bytes(L, vocab_size, block_size, chunk, k, sink)


def pulsar_maxidf_select(token_ids: torch.Tensor, vocab_size: int, block_size: int, chunk: int, k: int,
                         sink: int, want_df: bool = False, want_idf: bool = False, workspace=None,
                         status=None, out=None):
    """Max-IDF summary selection.  ``token_ids``: CUDA int32 [L] holding the uint32 ids.
    Returns a dict of CUDA tensors: sel_chunks [B,k], prefix_idx, prefix_len [B] (+ df, idf),
    B = ceil(L / block_size)."""
    lib = load_library()
    _need(token_ids, torch.int32, "token_ids")
    L = token_ids.numel()
    dev = token_ids.device
    B = -(-L // block_size) if block_size > 0 else 0          # the last block may be shorter
    if out is not None:                  # (sel_buf, prefix_idx, prefix_len) preallocated by the caller
        sel_buf, pidx, plen = out
    else:
        sel_buf = torch.empty(max(B, 0) * max(k, 0) + 4, dtype=torch.int32, device=dev)
        pidx = torch.empty(max(sink, 0) + max(B - 1, 0) * max(k, 0) * max(chunk, 0) + 4, dtype=torch.int32,
                           device=dev)
        plen = torch.empty(max(B, 1), dtype=torch.int32, device=dev)
    df = torch.empty(vocab_size, dtype=torch.int32, device=dev) if want_df else None
    idf = torch.empty(vocab_size, dtype=torch.float32, device=dev) if want_idf else None
    if workspace is None:
        workspace = _workspace(maxidf_select_workspace_bytes(L, vocab_size, block_size, chunk, k, sink), dev)
    rc = lib.pulsar_maxidf_select(_p(token_ids), L, vocab_size, block_size, chunk, k, sink, _p(sel_buf), _p(pidx),
                                  _p(plen), _p(df), _p(idf), _p(workspace), workspace.numel(), _p(status),
                                  _stream())
    _check("pulsar_maxidf_select", rc)
    n_pref = sink + max(B - 1, 0) * k * chunk
    sel = sel_buf[: B * k].view(B, k)
    out = dict(sel_chunks=sel, prefix_idx=pidx[:n_pref], prefix_len=plen[:B])
    if want_df:
        out["df"] = df
    if want_idf:
        out["idf"] = idf
    return out


def pulsar_maxidf_select_noalloc(token_ids: torch.Tensor, vocab_size: int, block_size: int, chunk: int, k: int,
                                 sink: int, sel_chunks: torch.Tensor, prefix_idx: torch.Tensor,
                                 prefix_len: torch.Tensor, status=None, df_out=None, idf_out=None):
    """Selection through the entry point that needs no workspace (its scratch is built into the
    library, 4 MiB per GPU).  The caller passes every buffer: token_ids int32 [L] in, and the
    outputs sel_chunks [B*k], prefix_idx [sink+(B-1)*k*chunk], prefix_len [B] (CUDA int32).
    ``df_out`` (int32 [vocab]) and ``idf_out`` (float32 [vocab]) optionally receive the tables.
    Raises PulsarError(PULSAR_ERR_WORKSPACE) if the problem does not fit the built-in scratch.
    Calls that may overlap on the GPU share that scratch and must be ordered by the caller."""
    lib = load_library()
    for t, n in ((token_ids, "token_ids"), (sel_chunks, "sel_chunks"), (prefix_idx, "prefix_idx"),
                 (prefix_len, "prefix_len")):
        _need(t, torch.int32, n)
    if df_out is not None:
        _need(df_out, torch.int32, "df_out")
    if idf_out is not None:
        _need(idf_out, torch.float32, "idf_out")
    rc = lib.pulsar_maxidf_select_noalloc(_p(token_ids), token_ids.numel(), vocab_size, block_size, chunk, k, sink,
                                          _p(sel_chunks), _p(prefix_idx), _p(prefix_len), _p(df_out), _p(idf_out),
                                          _p(status), _stream())
    _check("pulsar_maxidf_select_noalloc", rc)


SCORE_MODES = {"max_idf": 0, "tf_idf": 1, "bm25": 2, "type_token": 3}


def pulsar_chunk_select(token_ids: torch.Tensor, vocab_size: int, block_size: int, chunk: int, k: int, sink: int,
                        score_mode, want_score: bool = False, workspace=None, status=None):
    """Selection under one of the chunk scores of the paper's Appendix C (``score_mode``: a key of
    SCORE_MODES or its number).  Returns a dict of CUDA tensors: sel_chunks [B,k], prefix_idx,
    prefix_len [B] and, if asked for, score [B,C] float64."""
    lib = load_library()
    _need(token_ids, torch.int32, "token_ids")
    mode = SCORE_MODES.get(score_mode, score_mode)
    L = token_ids.numel()
    dev = token_ids.device
    B = -(-L // block_size) if block_size > 0 else 0
    C = -(-block_size // chunk) if chunk > 0 else 0
    sel_buf = torch.empty(max(B, 0) * max(k, 0) + 4, dtype=torch.int32, device=dev)
    pidx = torch.empty(max(sink, 0) + max(B - 1, 0) * max(k, 0) * max(chunk, 0) + 4, dtype=torch.int32, device=dev)
    plen = torch.empty(max(B, 1), dtype=torch.int32, device=dev)
    score = torch.empty((max(B, 1), max(C, 1)), dtype=torch.float64, device=dev) if want_score else None
    if workspace is None:
        workspace = _workspace(lib.pulsar_chunk_select_workspace_bytes(L, vocab_size, block_size, chunk, k, sink,
                                                                       int(mode)), dev)
    rc = lib.pulsar_chunk_select(_p(token_ids), L, vocab_size, block_size, chunk, k, sink, int(mode), _p(sel_buf),
                                 _p(pidx), _p(plen), _p(score), _p(workspace), workspace.numel(), _p(status),
                                 _stream())
    _check("pulsar_chunk_select", rc)
    out = dict(sel_chunks=sel_buf[: B * k].view(B, k), prefix_idx=pidx[: sink + max(B - 1, 0) * k * chunk],
               prefix_len=plen[:B])
    if want_score:
        out["score"] = score
    return out


def phase1_workspace_bytes(L, Hq, Hkv, d, block_size, prefix_total) -> int:
    return load_library().pulsar_phase1_workspace_bytes(L, Hq, Hkv, d, block_size, prefix_total)


def pulsar_phase1_attn(Q, K, V, block_size: int, prefix_idx, prefix_len, softmax_scale: float = 0.0,
                       want_lse: bool = True, retain_copy: bool = False, out=None, lse_out=None, workspace=None,
                       status=None):
    """Phase-1 prefix-block attention.  Q [L,Hq,d], K,V [L,Hkv,d] CUDA bf16; prefix_idx,
    prefix_len CUDA int32.  Returns (O bf16 [L,Hq,d], LSE f32 [L,Hq] or None, K_ret, V_ret)."""
    lib = load_library()
    for t, n in ((Q, "Q"), (K, "K"), (V, "V")):
        _need(t, torch.bfloat16, n)
    _need(prefix_len, torch.int32, "prefix_len")
    _need(prefix_idx, torch.int32, "prefix_idx")
    L, Hq, d = Q.shape
    Hkv = K.shape[1]
    dev = Q.device
    prefix_total = prefix_idx.numel()
    O = torch.empty_like(Q) if out is None else out
    LSE = lse_out if lse_out is not None else (
        torch.empty((L, Hq), dtype=torch.float32, device=dev) if want_lse else None)
    K_ret = torch.empty_like(K) if retain_copy else None
    V_ret = torch.empty_like(V) if retain_copy else None
    if workspace is None:
        workspace = _workspace(phase1_workspace_bytes(L, Hq, Hkv, d, block_size, prefix_total), dev)
    rc = lib.pulsar_phase1_attn(_p(Q), _p(K), _p(V), L, Hq, Hkv, d, block_size,
                                _p(prefix_idx) if prefix_total > 0 else None, _p(prefix_len), prefix_total,
                                float(softmax_scale), _p(O), _p(LSE), _p(K_ret), _p(V_ret),
                                _p(workspace), workspace.numel(), _p(status), _stream())
    _check("pulsar_phase1_attn", rc)
    if not retain_copy:
        K_ret, V_ret = K, V          # the retained KV is the block's own rows of K and V
    return O, LSE, K_ret, V_ret


def pulsar_causal_varlen_attn(Q, K, V, cu_seqlens, softmax_scale: float = 0.0, want_lse: bool = True, out=None,
                              workspace=None, status=None):
    """Causal attention over sequences packed back to back (the assembled Phase-1 inputs of the
    paper's whole-model pass).  Q [T,Hq,d], K,V [T,Hkv,d] CUDA bf16; cu_seqlens: host sequence of
    n_seq+1 ascending row offsets.  Returns (O bf16 [T,Hq,d], LSE f32 [T,Hq] or None)."""
    lib = load_library()
    for t, n in ((Q, "Q"), (K, "K"), (V, "V")):
        _need(t, torch.bfloat16, n)
    T, Hq, d = Q.shape
    Hkv = K.shape[1]
    cu = (ctypes.c_int32 * len(cu_seqlens))(*[int(x) for x in cu_seqlens])
    O = torch.empty_like(Q) if out is None else out
    LSE = torch.empty((T, Hq), dtype=torch.float32, device=Q.device) if want_lse else None
    if workspace is None:
        workspace = _workspace(256, Q.device)
    rc = lib.pulsar_causal_varlen_attn(_p(Q), _p(K), _p(V), T, ctypes.cast(cu, ctypes.c_void_p), len(cu_seqlens) - 1,
                                       Hq, Hkv, d, float(softmax_scale), _p(O), _p(LSE), _p(workspace),
                                       workspace.numel(), _p(status), _stream())
    _check("pulsar_causal_varlen_attn", rc)
    return O, LSE


def phase2_choose_splits(nq, B, block_size, Hq, Hkv, d) -> int:
    return load_library().pulsar_phase2_choose_splits(nq, B, block_size, Hq, Hkv, d)


def phase2_workspace_bytes(nq, B, block_size, Hq, Hkv, d, n_splits=0) -> int:
    return load_library().pulsar_phase2_workspace_bytes(nq, B, block_size, Hq, Hkv, d, n_splits)


def pulsar_phase2_attn(Qq, Kblocks, Vblocks, n_blocks: int, block_size: int, softmax_scale: float = 0.0,
                       n_splits: int = 0, want_partials: bool = False, out=None, lse_out=None, workspace=None,
                       status=None, partials=None):
    """Phase-2 query attention with exact LSE merge.  Qq [nq,Hq,d], K/V [n_blocks*block_size,Hkv,d]
    CUDA bf16.  Returns (O bf16 [nq,Hq,d], LSE f32 [nq,Hq]) and, with ``want_partials``
    (needs n_splits > 0), also (part_O f32 [J,nq,Hq,d], part_LSE f32 [J,nq,Hq]); ``partials`` may
    give those two tensors preallocated."""
    lib = load_library()
    for t, n in ((Qq, "Qq"), (Kblocks, "Kblocks"), (Vblocks, "Vblocks")):
        _need(t, torch.bfloat16, n)
    nq, Hq, d = Qq.shape
    Hkv = Kblocks.shape[-2]
    dev = Qq.device
    O = torch.empty_like(Qq) if out is None else out
    LSE = lse_out if lse_out is not None else torch.empty((nq, Hq), dtype=torch.float32, device=dev)
    pO = pL = None
    if partials is not None:
        pO, pL = partials
        want_partials = True
        _need(pO, torch.float32, "part_O")
        _need(pL, torch.float32, "part_LSE")
    elif want_partials:
        pO = torch.empty((n_splits, nq, Hq, d), dtype=torch.float32, device=dev)
        pL = torch.empty((n_splits, nq, Hq), dtype=torch.float32, device=dev)
    if workspace is None:
        workspace = _workspace(phase2_workspace_bytes(nq, n_blocks, block_size, Hq, Hkv, d, n_splits), dev)
    rc = lib.pulsar_phase2_attn(_p(Qq), nq, _p(Kblocks), _p(Vblocks), n_blocks, block_size, Hq, Hkv, d,
                                float(softmax_scale), n_splits, _p(O), _p(LSE), _p(pO), _p(pL),
                                _p(workspace), workspace.numel(), _p(status), _stream())
    _check("pulsar_phase2_attn", rc)
    return (O, LSE, pO, pL) if want_partials else (O, LSE)


def pulsar_phase2_generate_step(Qnew, Knew, Vnew, Kblocks, Vblocks, n_blocks: int, block_size: int, Kgen, Vgen,
                                gen_len: int, softmax_scale: float = 0.0, n_splits: int = 0, out=None,
                                workspace=None, status=None):
    """One generation step: append Knew/Vnew to the generation shard (rows gen_len..), then the
    n_new tokens attend to all context KV and, causally, to the shard; merged exactly.
    Qnew [n_new,Hq,d], Knew/Vnew [n_new,Hkv,d], Kgen/Vgen [capacity,Hkv,d] CUDA bf16 (updated in
    place).  Returns (O bf16 [n_new,Hq,d], LSE f32 [n_new,Hq]); the caller adds n_new to gen_len."""
    lib = load_library()
    for t, n in ((Qnew, "Qnew"), (Knew, "Knew"), (Vnew, "Vnew"), (Kblocks, "Kblocks"), (Vblocks, "Vblocks"),
                 (Kgen, "Kgen"), (Vgen, "Vgen")):
        _need(t, torch.bfloat16, n)
    n_new, Hq, d = Qnew.shape
    Hkv = Kblocks.shape[-2]
    if n_splits == 0:
        n_splits = phase2_choose_splits(n_new, n_blocks, block_size, Hq, Hkv, d)
    O = torch.empty_like(Qnew) if out is None else out
    LSE = torch.empty((n_new, Hq), dtype=torch.float32, device=Qnew.device)
    if workspace is None:
        workspace = _workspace(lib.pulsar_phase2_generate_workspace_bytes(n_new, n_blocks, block_size, Hq, Hkv, d,
                                                                          n_splits), Qnew.device)
    rc = lib.pulsar_phase2_generate_step(_p(Qnew), _p(Knew), _p(Vnew), n_new, _p(Kblocks), _p(Vblocks), n_blocks,
                                         block_size, _p(Kgen), _p(Vgen), gen_len, Kgen.shape[0], Hq, Hkv, d,
                                         float(softmax_scale), n_splits, _p(O), _p(LSE), _p(workspace),
                                         workspace.numel(), _p(status), _stream())
    _check("pulsar_phase2_generate_step", rc)
    return O, LSE


def pulsar_lse_merge(part_O, part_LSE, want_lse: bool = True):
    """Merge partials: part_O f32 [J,rows,d], part_LSE f32 [J,rows] -> (O bf16 [rows,d], LSE f32 [rows])."""
    lib = load_library()
    _need(part_O, torch.float32, "part_O")
    _need(part_LSE, torch.float32, "part_LSE")
    J, rows, d = part_O.shape
    O = torch.empty((rows, d), dtype=torch.bfloat16, device=part_O.device)
    LSE = torch.empty(rows, dtype=torch.float32, device=part_O.device) if want_lse else None
    rc = lib.pulsar_lse_merge(_p(part_O), _p(part_LSE), J, rows, d, _p(O), _p(LSE), _stream())
    _check("pulsar_lse_merge", rc)
    return O, LSE


def pulsar_lse_merge_strided(part_O, part_LSE, n_parts: int, part_stride_O: int, part_stride_LSE: int, rows: int,
                             d: int, out, lse_out=None):
    """Merge ``n_parts`` partials that start ``part_stride_*`` floats apart (part_O, part_LSE: CUDA
    float32 tensors or views whose data pointer is part 0).  ``out``: [rows, d] float32 (the result
    stays a partial) or bf16."""
    lib = load_library()
    _need(part_O, torch.float32, "part_O")
    _need(part_LSE, torch.float32, "part_LSE")
    if out.dtype not in (torch.float32, torch.bfloat16):
        raise TypeError("out must be float32 or bfloat16")
    rc = lib.pulsar_lse_merge_strided(_p(part_O), _p(part_LSE), n_parts, part_stride_O, part_stride_LSE, rows, d,
                                      _p(out), 1 if out.dtype == torch.float32 else 0, _p(lse_out), _stream())
    _check("pulsar_lse_merge_strided", rc)
    return out, lse_out


def pulsar_pack_summary_kv(K, V, block_size: int, sel_chunks, block_ids, n_blocks: int, chunk: int, k: int,
                           sink: int, K_send, V_send, status=None):
    """This GPU's contribution to the prefix exchange: K, V [n_local*block_size, Hkv, d] bf16 (its
    blocks), sel_chunks int32 [n_blocks, k], block_ids int32 [n_local] (CUDA) -> K_send, V_send
    [sink + n_local*k*chunk, Hkv, d] bf16."""
    lib = load_library()
    for t, n in ((K, "K"), (V, "V"), (K_send, "K_send"), (V_send, "V_send")):
        _need(t, torch.bfloat16, n)
    _need(sel_chunks, torch.int32, "sel_chunks")
    _need(block_ids, torch.int32, "block_ids")
    Hkv, d = K.shape[-2], K.shape[-1]
    rc = lib.pulsar_pack_summary_kv(_p(K), _p(V), block_ids.numel(), block_size, Hkv, d, _p(sel_chunks), _p(block_ids),
                                    n_blocks, chunk, k, sink, _p(K_send), _p(V_send), _p(status), _stream())
    _check("pulsar_pack_summary_kv", rc)


def pulsar_gather_kv_rows(K, V, idx, K_out, V_out, status=None):
    """K_out[j] = K[idx[j]], V_out[j] = V[idx[j]] (rows of [rows, Hkv, d] bf16; idx CUDA int32)."""
    lib = load_library()
    for t, n in ((K, "K"), (V, "V"), (K_out, "K_out"), (V_out, "V_out")):
        _need(t, torch.bfloat16, n)
    _need(idx, torch.int32, "idx")
    rc = lib.pulsar_gather_kv_rows(_p(K), _p(V), K.shape[0], K.shape[-2], K.shape[-1], _p(idx), idx.numel(),
                                   _p(K_out), _p(V_out), _p(status), _stream())
    _check("pulsar_gather_kv_rows", rc)


def pulsar_phase1_attn_sharded(Q, K, V, block_size: int, K_prefix, V_prefix, prefix_len_local,
                               softmax_scale: float = 0.0, want_lse: bool = True, out=None, lse_out=None,
                               workspace=None, status=None):
    """Phase-1 attention over this GPU's blocks (Q [L_local,Hq,d], K,V [L_local,Hkv,d]) with the
    prefix K/V rows already in local memory in prefix-list order (K_prefix, V_prefix
    [prefix_total,Hkv,d]); prefix_len_local int32 [L_local/block_size].  Returns (O, LSE)."""
    lib = load_library()
    for t, n in ((Q, "Q"), (K, "K"), (V, "V")):
        _need(t, torch.bfloat16, n)
    _need(prefix_len_local, torch.int32, "prefix_len_local")
    L, Hq, d = Q.shape
    Hkv = K.shape[1]
    prefix_total = 0 if K_prefix is None else K_prefix.shape[0]
    if prefix_total:
        _need(K_prefix, torch.bfloat16, "K_prefix")
        _need(V_prefix, torch.bfloat16, "V_prefix")
    O = torch.empty_like(Q) if out is None else out
    LSE = lse_out if lse_out is not None else (
        torch.empty((L, Hq), dtype=torch.float32, device=Q.device) if want_lse else None)
    if workspace is None:
        workspace = _workspace(256, Q.device)
    rc = lib.pulsar_phase1_attn_sharded(_p(Q), _p(K), _p(V), L, Hq, Hkv, d, block_size,
                                        _p(K_prefix) if prefix_total else None,
                                        _p(V_prefix) if prefix_total else None, prefix_total,
                                        _p(prefix_len_local), float(softmax_scale), _p(O), _p(LSE), _p(workspace),
                                        workspace.numel(), _p(status), _stream())
    _check("pulsar_phase1_attn_sharded", rc)
    return O, LSE


POSITION_MODES = {"sparse": 0, "contiguous": 1}


def pulsar_assemble_positions(prefix_idx, prefix_len, n_blocks: int, block_size: int, total: int, mode="sparse",
                              status=None):
    """Position ids (CUDA int32 [total]) of the assembled Phase-1 inputs stored back to back;
    ``total`` = sum_i (prefix_len[i] + block_size), which the caller knows from the layout."""
    lib = load_library()
    _need(prefix_len, torch.int32, "prefix_len")
    _need(prefix_idx, torch.int32, "prefix_idx")
    pos = torch.empty(max(total, 1), dtype=torch.int32, device=prefix_len.device)
    n_pref = prefix_idx.numel()
    rc = lib.pulsar_assemble_positions(_p(prefix_idx) if n_pref else None, _p(prefix_len), n_pref, n_blocks,
                                       block_size, POSITION_MODES.get(mode, mode), _p(pos), total, _p(status),
                                       _stream())
    _check("pulsar_assemble_positions", rc)
    return pos[:total]


def pulsar_rope_apply(X, positions, theta: float = 500000.0, out=None, status=None):
    """Rotary embedding of X [rows,H,d] CUDA bf16 at ``positions`` (CUDA int32 [rows]); rotate-half
    pairing.  ``out`` may be X itself (in place)."""
    lib = load_library()
    _need(X, torch.bfloat16, "X")
    _need(positions, torch.int32, "positions")
    rows, H, d = X.shape
    if positions.numel() != rows:
        raise ValueError("one position id per row")
    Y = torch.empty_like(X) if out is None else out
    rc = lib.pulsar_rope_apply(_p(X), _p(Y), rows, H, d, _p(positions), float(theta), _p(status), _stream())
    _check("pulsar_rope_apply", rc)
    return Y


def pulsar_rope_apply_qk(Q, K, positions, theta: float = 500000.0, q_out=None, k_out=None, status=None):
    """Rotary embedding of Q [rows,Hq,d] and K [rows,Hkv,d] (CUDA bf16) in one launch; the outputs
    default to new tensors and may be the inputs themselves."""
    lib = load_library()
    _need(Q, torch.bfloat16, "Q")
    _need(K, torch.bfloat16, "K")
    _need(positions, torch.int32, "positions")
    rows, Hq, d = Q.shape
    if K.shape[0] != rows or K.shape[2] != d or positions.numel() != rows:
        raise ValueError("Q, K and positions must cover the same rows and head size")
    Qo = torch.empty_like(Q) if q_out is None else q_out
    Ko = torch.empty_like(K) if k_out is None else k_out
    rc = lib.pulsar_rope_apply_qk(_p(Q), _p(Qo), Hq, _p(K), _p(Ko), K.shape[1], rows, d, _p(positions), float(theta),
                                  _p(status), _stream())
    _check("pulsar_rope_apply_qk", rc)
    return Qo, Ko


def pulsar_lse_merge_peers(part_ptrs, rows_total: int, row_begin: int, rows: int, d: int, out, lse_out=None):
    """Merge rows [row_begin, row_begin+rows) of the partials at the device addresses ``part_ptrs``
    (ints: this GPU's buffers or peer-mapped ones, each laid out [rows_total*d | rows_total] float32).
    ``out`` [rows, d] float32 or bf16 on the current device."""
    lib = load_library()
    n = len(part_ptrs)
    table = (ctypes.c_void_p * n)(*[ctypes.c_void_p(int(p)) for p in part_ptrs])
    rc = lib.pulsar_lse_merge_peers(ctypes.cast(table, ctypes.c_void_p), n, rows_total, row_begin, rows, d, _p(out),
                                    1 if out.dtype == torch.float32 else 0, _p(lse_out), _stream())
    _check("pulsar_lse_merge_peers", rc)
    return out, lse_out


def pulsar_retain_block_kv(K, V, cu_seqlens, block_size: int):
    """The retained KV of assembled inputs: the last ``block_size`` rows of every input.  K, V
    [total_rows,Hkv,d] CUDA bf16, cu_seqlens a host sequence.  Returns (K_ret, V_ret) [n_seq*block_size,Hkv,d]."""
    lib = load_library()
    _need(K, torch.bfloat16, "K")
    _need(V, torch.bfloat16, "V")
    cu = (ctypes.c_int32 * len(cu_seqlens))(*[int(x) for x in cu_seqlens])
    n_seq = len(cu_seqlens) - 1
    Kr = torch.empty((n_seq * block_size,) + tuple(K.shape[1:]), dtype=torch.bfloat16, device=K.device)
    Vr = torch.empty_like(Kr)
    rc = lib.pulsar_retain_block_kv(_p(K), _p(V), K.shape[0], ctypes.cast(cu, ctypes.c_void_p), n_seq, block_size,
                                    K.shape[1], K.shape[2], _p(Kr), _p(Vr), _stream())
    _check("pulsar_retain_block_kv", rc)
    return Kr, Vr
