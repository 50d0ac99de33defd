"""Binding of the attention-block entry points (include/resq_kv.h): argument marshalling only."""
from __future__ import annotations

import ctypes

from . import ERR_CUDA, ERR_INDEX, OK, ResqError, _check, _ptr, _stream, lib  # noqa: F401

KV_BLOCK, KV_BLOCK_BYTES = 32, 5632
KV_EXPORTS = ["resq_kv_block_bytes", "resq_kv_cache_bytes", "resq_uc_quantize", "resq_query_project", "resq_kv_append", "resq_qkv_project_append",
              "resq_attention_workspace_bytes", "resq_attention_decode", "resq_attention_queries_workspace_bytes",
              "resq_attention_queries", "resq_attention_prefill"]


class KvCacheStruct(ctypes.Structure):
    _fields_ = [("n_seqs", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32), ("d_head", ctypes.c_int32),
                ("capacity", ctypes.c_int32), ("data", ctypes.c_void_p)]


_vp, _sz, _i, _i64 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_int64
_cp = ctypes.POINTER(KvCacheStruct)
lib.resq_kv_block_bytes.restype = _sz
lib.resq_kv_block_bytes.argtypes = [_i]
lib.resq_kv_cache_bytes.restype = _sz
lib.resq_kv_cache_bytes.argtypes = [_i, _i, _i, _i]
lib.resq_uc_quantize.argtypes = [_vp, _i, _vp, _vp, _vp]
lib.resq_query_project.argtypes = [_vp, _i64, _i, _vp, _vp, _vp, _vp]
lib.resq_kv_append.argtypes = [_cp, _vp, _vp, _i64, _vp, _vp, _vp, _vp, _vp]
lib.resq_qkv_project_append.argtypes = [_cp, _vp, _i, _vp, _vp, _vp, _i64, _vp, _vp, _vp, _vp, _vp]
lib.resq_attention_workspace_bytes.restype = _sz
lib.resq_attention_workspace_bytes.argtypes = [_i, _i, _i, _i]
lib.resq_attention_decode.argtypes = [_cp, _vp, _i, _vp, _vp, _vp, _sz, _vp]
lib.resq_attention_queries_workspace_bytes.restype = _sz
lib.resq_attention_queries_workspace_bytes.argtypes = [_i, _i, _i, _i]
lib.resq_attention_queries.argtypes = [_cp, _vp, _i, _i, _vp, _vp, _vp, _vp, _sz, _vp]
lib.resq_attention_prefill.argtypes = [_cp, _vp, _i, _i, _i, _i, _vp, _vp]


class KvCache:
    """Geometry plus the caller's buffer (a torch uint8 tensor used as device memory)."""

    def __init__(self, n_seqs: int, n_kv_heads: int, capacity: int, d_head: int = 128, device="cuda", data=None):
        import torch
        self.n_seqs, self.n_kv_heads, self.capacity, self.d_head = n_seqs, n_kv_heads, capacity, d_head
        nbytes = int(lib.resq_kv_cache_bytes(n_seqs, n_kv_heads, d_head, capacity))
        if nbytes == 0:
            raise ResqError(2, "resq_kv_cache_bytes")
        self.data = torch.empty(nbytes, dtype=torch.uint8, device=device) if data is None else data
        self.c = KvCacheStruct(n_seqs, n_kv_heads, d_head, capacity, self.data.data_ptr())

    @property
    def nbytes(self) -> int:
        return self.data.numel()


def resq_uc_quantize(W_C):
    """W_C = U_C^T fp32 [128][128] -> (codes int8 [128][128], scales fp32 [128])."""
    import torch
    d = W_C.shape[0]
    wq = torch.empty((d, d), dtype=torch.int8, device=W_C.device)
    s_u = torch.empty(d, dtype=torch.float32, device=W_C.device)
    _check(lib.resq_uc_quantize(_ptr(W_C), d, _ptr(wq), _ptr(s_u), _stream()), "resq_uc_quantize")
    return wq, s_u


def resq_query_project(q, wq, s_u, q_out):
    """q bf16 [..., 128] -> q_out half of the same shape."""
    rows = q.numel() // q.shape[-1]
    _check(lib.resq_query_project(_ptr(q), rows, q.shape[-1], _ptr(wq), _ptr(s_u), _ptr(q_out), _stream()),
           "resq_query_project")


def resq_kv_append(cache: KvCache, k, v, seq_ids, positions, wq, s_u):
    """k, v bf16 [T][n_kv_heads][128]; seq_ids, positions int32 [T]."""
    _check(lib.resq_kv_append(ctypes.byref(cache.c), _ptr(k), _ptr(v), k.shape[0], _ptr(seq_ids), _ptr(positions),
                              _ptr(wq), _ptr(s_u), _stream()), "resq_kv_append")


def resq_qkv_project_append(cache: KvCache, q, q_out, k, v, seq_ids, positions, wq, s_u):
    """q bf16 [T][n_q_heads][128] -> q_out half; k, v bf16 [T][n_kv_heads][128] appended; one launch."""
    _check(lib.resq_qkv_project_append(ctypes.byref(cache.c), _ptr(q), q.shape[1], _ptr(q_out), _ptr(k), _ptr(v),
                                       k.shape[0], _ptr(seq_ids), _ptr(positions), _ptr(wq), _ptr(s_u), _stream()),
           "resq_qkv_project_append")


def attention_workspace(cache: KvCache, n_q_heads: int):
    import torch
    n = int(lib.resq_attention_workspace_bytes(cache.n_seqs, n_q_heads, cache.n_kv_heads, cache.d_head))
    if n == 0:
        raise ResqError(2, "resq_attention_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=cache.data.device)


def resq_attention_decode(cache: KvCache, q16, seq_lens, out, workspace):
    """q16 half [n_seqs][n_q_heads][128], seq_lens int32 [n_seqs], out fp32 [n_seqs][n_q_heads][128]."""
    _check(lib.resq_attention_decode(ctypes.byref(cache.c), _ptr(q16), q16.shape[1], _ptr(seq_lens), _ptr(out),
                                     _ptr(workspace), workspace.numel(), _stream()), "resq_attention_decode")


def resq_attention_queries(cache: KvCache, q16, q_seq, q_len, out, workspace=None):
    """q16 half [n_queries][n_q_heads][128]; query row i attends the first q_len[i] positions of cache sequence
    q_seq[i] (int32 tensors); out fp32 of q16's shape.  Allocates the scratch if none is given."""
    import torch
    n, hq = q16.shape[0], q16.shape[1]
    if workspace is None:
        nbytes = int(lib.resq_attention_queries_workspace_bytes(n, hq, cache.n_kv_heads, cache.d_head))
        if nbytes == 0:
            raise ResqError(2, "resq_attention_queries_workspace_bytes")
        workspace = torch.empty(nbytes, dtype=torch.uint8, device=cache.data.device)
    _check(lib.resq_attention_queries(ctypes.byref(cache.c), _ptr(q16), hq, n, _ptr(q_seq), _ptr(q_len), _ptr(out),
                                      _ptr(workspace), workspace.numel(), _stream()), "resq_attention_queries")


def resq_attention_prefill(cache: KvCache, q16, seq: int, pos0: int, out):
    """q16 half [T][n_q_heads][128]: token t, at position pos0 + t of cache sequence `seq`, attends positions
    0 .. pos0 + t (already appended); out fp32 of q16's shape."""
    _check(lib.resq_attention_prefill(ctypes.byref(cache.c), _ptr(q16), q16.shape[1], int(seq), int(pos0), q16.shape[0],
                                      _ptr(out), _stream()), "resq_attention_prefill")
