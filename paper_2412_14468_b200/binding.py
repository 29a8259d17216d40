"""Thin ctypes binding over libhashattn.so: argument marshalling only.

Every function has the name and semantics of the C entry point declared in include/hashattn.h;
tensors are torch tensors used purely as device (or pinned host) memory handles.  There is no
fallback: if the CUDA library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libhashattn.so")

HA_OK = 0
HA_ERR_INVALID_ARG, HA_ERR_UNSUPPORTED, HA_ERR_WORKSPACE, HA_ERR_CUDA, HA_ERR_STATIC_LIMIT = 1, 2, 3, 4, 5
HA_DEV_BAD_INDEX, HA_DEV_TIMEOUT = 1, 2
HIST_BINS = 33

EXPORTS = [
    "ha_workspace_bytes", "ha_workspace_init", "ha_encode", "ha_encode_prefill", "ha_score_topk", "ha_gather_attn",
    "ha_gather_attn_paged", "ha_sparse_decode_paged",
    "ha_gather_attn_static", "ha_dense_decode", "ha_sparse_decode", "ha_sparse_decode_host", "ha_read_device_status",
    "ha_score_wide", "ha_inner_products", "ha_sparse_decode_paged_host", "ha_score_topk_sum",
    "ha_score_topk_per_head", "ha_gather_attn_per_head", "ha_sparse_decode_pipelined",
    "ha_encode_wide", "ha_workspace_bytes_wide", "ha_score_topk_wide",
    "ha_score_topk_paged", "ha_score_topk_per_head_paged", "ha_gather_attn_per_head_paged", "ha_encode_append_paged",
    "ha_sparse_decode_paged_codes",
    "ha_kernel_launches", "ha_status_string", "ha_version",
]


class ha_shape(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("sm_scale", C.c_float), ("n_sink", C.c_int32), ("n_local", C.c_int32)]


class ha_mapping(C.Structure):
    _fields_ = [("n_kv_heads", C.c_int32), ("in_dim", C.c_int32), ("hid_dim", C.c_int32), ("n_bits", C.c_int32),
                ("w1", C.c_void_p), ("w2", C.c_void_p), ("w3", C.c_void_p),
                ("b1", C.c_void_p), ("b2", C.c_void_p), ("b3", C.c_void_p)]


class ha_tensor(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("stride_b", C.c_int64), ("stride_h", C.c_int64), ("stride_n", C.c_int64)]


class HashAttnError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        super().__init__(f"{fn} failed: {status_string(status)} (status {status})")


_lib = None


def lib() -> C.CDLL:
    """Load libhashattn.so (built by paper_2412_14468_b200/build.py).  Raises if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: run `python -m paper_2412_14468_b200.build` "
                               "(nvcc, sm_100a); this package has no CPU fallback")
        L = C.CDLL(LIB_PATH)
        P, I32, I64, SZ = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
        L.ha_workspace_bytes.restype = SZ
        L.ha_workspace_bytes.argtypes = [P, I32, I32]
        L.ha_workspace_init.argtypes = [P, SZ, P]
        L.ha_encode.argtypes = [P, I32, P, I32, I32, I32, P, I64, I64, P, P]
        L.ha_encode_prefill.argtypes = [P, I32, P, I32, I32, I32, P, I64, I64, I32, P, P]
        L.ha_score_topk.argtypes = [P, P, P, I64, I64, P, P, I32, I32, I32, P, I64, I64, P, P, P, SZ, P]
        L.ha_score_topk_sum.argtypes = [P, P, P, I64, I64, P, P, I32, I32, P, I64, I64, P, P, P]
        L.ha_score_topk_per_head.argtypes = [P, P, P, I64, I64, P, P, I32, I32, P, I64, I64, P, P, P]
        L.ha_gather_attn_per_head.argtypes = [P, P, P, P, P, P, I64, I64, P, I32, P, P, P, SZ, P]
        L.ha_gather_attn.argtypes = [P, P, P, P, P, P, I64, I64, P, I32, P, P, P, SZ, P]
        L.ha_gather_attn_paged.argtypes = [P, P, P, P, P, I64, I32, P, P, I64, I64, P, I32, P, P, P, SZ, P]
        L.ha_gather_attn_static.argtypes = [P, P, P, P, P, P, I64, I64, P, I32, P, P, P]
        L.ha_dense_decode.argtypes = [P, P, P, P, P, I32, P, P, P, SZ, P]
        L.ha_sparse_decode.argtypes = [P, P, P, P, P, P, P, P, I64, I64, P, P, I32, I32, I32, P, P, I64, I64, P,
                                       P, P, P, SZ, P]
        L.ha_sparse_decode_pipelined.argtypes = L.ha_sparse_decode.argtypes
        L.ha_sparse_decode_pipelined.restype = C.c_int
        L.ha_sparse_decode_paged.argtypes = [P, P, P, P, P, P, P, P, I64, I32, P, I64, I64, P, P, I32, I32, I32, P, P, I64, I64,
                                             P, P, P, P, SZ, P]
        L.ha_sparse_decode_host.argtypes = [P, P, P, P, P, P, P, P, P, I64, I64, P, P, I32, I32, I32, P, I64, I64,
                                            P, P, P, SZ, P]
        L.ha_read_device_status.argtypes = [P, P, P]
        L.ha_sparse_decode_paged_host.argtypes = [P, P, P, P, P, P, P, P, P, I64, I32, P, I64, I64, P, P, I32, I32, I32, P,
                                                  I64, I64, P, P, P, SZ, P]
        L.ha_score_wide.argtypes = [P, P, I64, I32, P, P]
        L.ha_score_topk_paged.argtypes = [P, P, P, I64, I64, P, I64, I32, P, P, I32, I32, I32, P, I64, I64, P, P, P, SZ, P]
        L.ha_score_topk_per_head_paged.argtypes = L.ha_score_topk_paged.argtypes
        L.ha_gather_attn_per_head_paged.argtypes = L.ha_gather_attn_paged.argtypes
        L.ha_encode_append_paged.argtypes = [P, P, I32, P, I64, I64, P, I64, I32, P, P]
        L.ha_sparse_decode_paged_codes.argtypes = [P, P, P, P, P, P, P, P, I64, I64, P, I64, I32, P, P, I32, I32, I32, P, P,
                                                   I64, I64, P, P, P, P, SZ, P]
        for fn in ("ha_score_topk_paged", "ha_score_topk_per_head_paged", "ha_gather_attn_per_head_paged",
                   "ha_encode_append_paged", "ha_sparse_decode_paged_codes"):
            getattr(L, fn).restype = C.c_int
        L.ha_encode_wide.argtypes = [P, I32, P, I32, I32, I32, P, I64, I64, P, P]
        L.ha_encode_wide.restype = C.c_int
        L.ha_workspace_bytes_wide.restype = SZ
        L.ha_workspace_bytes_wide.argtypes = [P, I32]
        L.ha_score_topk_wide.argtypes = [P, I32, P, P, I64, I64, P, P, I32, I32, I32, P, I64, I64, P, P, P, SZ, P]
        L.ha_score_topk_wide.restype = C.c_int
        L.ha_inner_products.argtypes = [P, P, I64, I64, P, P]
        L.ha_kernel_launches.restype = C.c_uint64
        L.ha_status_string.restype = C.c_char_p
        L.ha_status_string.argtypes = [C.c_int]
        L.ha_version.restype = C.c_char_p
        for fn in ("ha_workspace_init", "ha_encode", "ha_score_topk", "ha_gather_attn", "ha_gather_attn_static", "ha_dense_decode",
                   "ha_sparse_decode", "ha_sparse_decode_host", "ha_read_device_status", "ha_score_wide",
                   "ha_inner_products", "ha_sparse_decode_paged_host", "ha_sparse_decode_paged", "ha_gather_attn_paged",
                   "ha_encode_prefill", "ha_score_topk_sum", "ha_score_topk_per_head", "ha_gather_attn_per_head"):
            getattr(L, fn).restype = C.c_int
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().ha_status_string(int(status)).decode()


def ha_version() -> str:
    return lib().ha_version().decode()


def ha_score_wide(q_code: torch.Tensor, k_codes: torch.Tensor, n_bits: int, scores: torch.Tensor, stream=None) -> None:
    """q_code int64 [n_bits/64]; k_codes int64 [n, n_bits/64] (the 64-bit words of the signatures); scores int16 [n]."""
    _dev(q_code, torch.int64, "q_code"); _dev(k_codes, torch.int64, "k_codes"); _dev(scores, torch.int16, "scores")
    assert k_codes.is_contiguous() and q_code.is_contiguous() and scores.is_contiguous()
    n = k_codes.shape[0]
    assert k_codes.dim() == 2 and k_codes.shape[1] * 64 == n_bits == q_code.numel() * 64 and scores.numel() == n
    _check("ha_score_wide", lib().ha_score_wide(q_code.data_ptr(), k_codes.data_ptr(), n, n_bits, scores.data_ptr(),
                                                _stream(stream)))


class MappingWide:
    """Device-resident weights of one side's mapping networks with a last layer of 128 x n_bits (64 .. 512)."""

    def __init__(self, weights: Dict[str, torch.Tensor]):
        self.t = {k: _dev(weights[k], torch.bfloat16, k).contiguous() for k in ("w1", "w2", "w3")}
        for k in ("b1", "b2", "b3"):
            b = weights.get(k)
            self.t[k] = None if b is None else _dev(b, torch.float32, k).contiguous()
        hkv, n_bits = self.t["w1"].shape[0], self.t["w3"].shape[2]
        assert tuple(self.t["w1"].shape) == (hkv, 128, 128) and tuple(self.t["w2"].shape) == (hkv, 128, 128)
        assert tuple(self.t["w3"].shape) == (hkv, 128, n_bits)
        self.n_bits = n_bits
        self.struct = ha_mapping(hkv, 128, 128, n_bits, _ptr(self.t["w1"]), _ptr(self.t["w2"]), _ptr(self.t["w3"]),
                                 _ptr(self.t["b1"]), _ptr(self.t["b2"]), _ptr(self.t["b3"]))

    @property
    def ref(self):
        return C.byref(self.struct)


def ha_encode_wide(mapping: "MappingWide", heads_per_kv: int, x: torch.Tensor, codes: torch.Tensor,
                   slot: Optional[torch.Tensor] = None, stream=None) -> None:
    """x: bf16 [B,H,T,128] (or [B,H,128]); codes: int64 [B,H,>=T,n_bits/64] (the packed 64-bit words, contiguous per token)."""
    xt = make_tensor(x)
    B, H = x.shape[0], x.shape[1]
    T = 1 if x.dim() == 3 else x.shape[2]
    _dev(codes, torch.int64, "codes")
    assert codes.dim() == 4 and codes.stride(3) == 1 and codes.stride(2) == codes.shape[3] == mapping.n_bits // 64
    _check("ha_encode_wide", lib().ha_encode_wide(mapping.ref, heads_per_kv, C.byref(xt), B, H, T, codes.data_ptr(),
                                                  codes.stride(0), codes.stride(1), _ptr(slot), _stream(stream)))


def ha_workspace_bytes_wide(shape: ha_shape, max_seq_len: int) -> int:
    n = int(lib().ha_workspace_bytes_wide(C.byref(shape), max_seq_len))
    if n == 0:
        raise HashAttnError("ha_workspace_bytes_wide", HA_ERR_UNSUPPORTED)
    return n


def alloc_workspace_wide(shape: ha_shape, max_seq_len: int, device="cuda") -> torch.Tensor:
    return torch.empty(ha_workspace_bytes_wide(shape, max_seq_len), dtype=torch.uint8, device=device)


def ha_score_topk_wide(shape: ha_shape, n_bits: int, q_codes, k_codes, seq_lens, k_per_seq, k_uniform: int, max_seq_len: int,
                       k_max: int, idx, count, workspace, hist_out=None, stream=None) -> None:
    """q_codes int64 [B,Hq,W]; k_codes int64 [B,Hkv,N,W] (W = n_bits/64 words per token); idx int32 [B,Hkv,k_max]."""
    _dev(q_codes, torch.int64, "q_codes"); _dev(k_codes, torch.int64, "k_codes")
    assert q_codes.is_contiguous() and k_codes.dim() == 4 and k_codes.stride(3) == 1 and k_codes.stride(2) == k_codes.shape[3]
    p, n = _ws(workspace)
    _check("ha_score_topk_wide", lib().ha_score_topk_wide(
        C.byref(shape), n_bits, q_codes.data_ptr(), k_codes.data_ptr(), k_codes.stride(0), k_codes.stride(1),
        seq_lens.data_ptr(), _ptr(k_per_seq), k_uniform, max_seq_len, k_max, idx.data_ptr(), idx.stride(0), idx.stride(1),
        count.data_ptr(), _ptr(hist_out), p, n, _stream(stream)))


def ha_inner_products(q: torch.Tensor, K: torch.Tensor, dots: torch.Tensor, stream=None) -> None:
    """q bf16 [128]; K bf16 [n, 128] (row stride a multiple of 8 elements); dots fp32 [n]."""
    _dev(q, torch.bfloat16, "q"); _dev(K, torch.bfloat16, "K"); _dev(dots, torch.float32, "dots")
    assert K.dim() == 2 and K.shape[1] == 128 and K.stride(1) == 1 and q.numel() == 128 and dots.numel() == K.shape[0]
    _check("ha_inner_products", lib().ha_inner_products(q.data_ptr(), K.data_ptr(), K.shape[0], K.stride(0), dots.data_ptr(),
                                                        _stream(stream)))


def ha_kernel_launches() -> int:
    return int(lib().ha_kernel_launches())


def _check(fn: str, status: int) -> None:
    if status != HA_OK:
        raise HashAttnError(fn, status)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _dev(t: torch.Tensor, dtype, name: str) -> torch.Tensor:
    if not t.is_cuda or t.dtype != dtype:
        raise TypeError(f"{name}: expected a CUDA tensor of {dtype}, got {t.dtype} on {t.device}")
    return t


def make_shape(batch: int, n_q_heads: int, n_kv_heads: int, sm_scale: float, head_dim: int = 128,
               n_sink: int = 0, n_local: int = 0) -> ha_shape:
    """n_sink / n_local: tokens always in context in addition to the budget (SCORE + TOPK only)."""
    return ha_shape(batch, n_q_heads, n_kv_heads, head_dim, float(sm_scale), n_sink, n_local)


def make_tensor(t: torch.Tensor) -> ha_tensor:
    """bf16 [B,H,N,128] tensor (any strides with a contiguous last dim) -> ha_tensor."""
    _dev(t, torch.bfloat16, "tensor")
    if t.dim() == 3:                       # [B,H,128]: one token per head
        t = t.unsqueeze(2)
    if t.dim() != 4 or t.stride(3) != 1:
        raise ValueError("expected [B,H,N,128] with a contiguous last dimension")
    return ha_tensor(t.data_ptr(), t.stride(0), t.stride(1), t.stride(2) if t.shape[2] > 1 else max(t.stride(2), 128))


class Mapping:
    """Device-resident weights of one side's mapping networks + the ha_mapping struct over them."""

    def __init__(self, weights: Dict[str, torch.Tensor]):
        self.t = {}
        for k in ("w1", "w2", "w3"):
            self.t[k] = _dev(weights[k], torch.bfloat16, k).contiguous()
        for k in ("b1", "b2", "b3"):
            b = weights.get(k)
            self.t[k] = None if b is None else _dev(b, torch.float32, k).contiguous()
        hkv = self.t["w1"].shape[0]
        assert tuple(self.t["w1"].shape) == (hkv, 128, 128) and tuple(self.t["w2"].shape) == (hkv, 128, 128)
        assert tuple(self.t["w3"].shape) == (hkv, 128, 32)
        self.struct = ha_mapping(hkv, 128, 128, 32, _ptr(self.t["w1"]), _ptr(self.t["w2"]), _ptr(self.t["w3"]),
                                 _ptr(self.t["b1"]), _ptr(self.t["b2"]), _ptr(self.t["b3"]))

    @property
    def ref(self):
        return C.byref(self.struct)


def ha_workspace_bytes(shape: ha_shape, max_seq_len: int, max_k: int) -> int:
    n = int(lib().ha_workspace_bytes(C.byref(shape), max_seq_len, max_k))
    if n == 0:
        raise HashAttnError("ha_workspace_bytes", HA_ERR_UNSUPPORTED)
    return n


def ha_workspace_init(workspace: torch.Tensor, stream=None) -> None:
    _check("ha_workspace_init", lib().ha_workspace_init(workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                                       _stream(stream)))


def alloc_workspace(shape: ha_shape, max_seq_len: int, max_k: int, device="cuda") -> torch.Tensor:
    """Convenience for callers and tests: a uint8 workspace of the right size, already initialised."""
    ws = torch.empty(ha_workspace_bytes(shape, max_seq_len, max_k), dtype=torch.uint8, device=device)
    ha_workspace_init(ws)
    return ws


def _ws(ws: torch.Tensor):
    return ws.data_ptr(), ws.numel() * ws.element_size()


def ha_encode(mapping: Mapping, heads_per_kv: int, x: torch.Tensor, codes: torch.Tensor,
              slot: Optional[torch.Tensor] = None, stream=None) -> None:
    """x: bf16 [B,H,T,128] (or [B,H,128]); codes: int32/uint32-as-int32 [B,H,>=T] (last dim contiguous)."""
    xt = make_tensor(x)
    B, H = x.shape[0], x.shape[1]
    T = 1 if x.dim() == 3 else x.shape[2]
    _dev(codes, torch.int32, "codes")
    assert codes.dim() == 3 and codes.stride(2) == 1
    _check("ha_encode", lib().ha_encode(mapping.ref, heads_per_kv, C.byref(xt), B, H, T, codes.data_ptr(),
                                        codes.stride(0), codes.stride(1), _ptr(slot), _stream(stream)))


HA_PREFILL_TCGEN05, HA_PREFILL_MMA_SYNC = 0, 1


def ha_encode_prefill(mapping: Mapping, heads_per_kv: int, x: torch.Tensor, codes: torch.Tensor,
                      path: int = HA_PREFILL_TCGEN05, workspace: Optional[torch.Tensor] = None, stream=None) -> None:
    """Tensor-core ENCODE of whole prompts; x: bf16 [B,H,T,128]; codes: int32 [B,H,>=T] (last dim contiguous)."""
    xt = make_tensor(x)
    B, H = x.shape[0], x.shape[1]
    T = 1 if x.dim() == 3 else x.shape[2]
    _dev(codes, torch.int32, "codes")
    assert codes.dim() == 3 and codes.stride(2) == 1
    _check("ha_encode_prefill", lib().ha_encode_prefill(mapping.ref, heads_per_kv, C.byref(xt), B, H, T, codes.data_ptr(),
                                                        codes.stride(0), codes.stride(1), path, _ptr(workspace),
                                                        _stream(stream)))


def ha_score_topk(shape: ha_shape, q_codes, k_codes, seq_lens, k_per_seq, k_uniform: int, max_seq_len: int,
                  k_max: int, idx, count, workspace, hist_out=None, stream=None) -> None:
    """q_codes int32 [B,Hq]; k_codes int32 [B,Hkv,N]; idx int32 [B,Hkv,k_max]; count int32 [B,Hkv]."""
    p, n = _ws(workspace)
    _check("ha_score_topk", lib().ha_score_topk(
        C.byref(shape), q_codes.data_ptr(), k_codes.data_ptr(), k_codes.stride(0), k_codes.stride(1),
        seq_lens.data_ptr(), _ptr(k_per_seq), k_uniform, max_seq_len, k_max, idx.data_ptr(), idx.stride(0),
        idx.stride(1), count.data_ptr(), _ptr(hist_out), p, n, _stream(stream)))


def ha_score_topk_sum(shape: ha_shape, q_codes, k_codes, seq_lens, k_per_seq, k_uniform: int, k_max: int, idx, count,
                      hist_out=None, stream=None) -> None:
    """ha_score_topk with the per-head scores of a group added up (0 .. 32 G); hist_out int32 [B,Hkv,32 G + 1]."""
    _check("ha_score_topk_sum", lib().ha_score_topk_sum(
        C.byref(shape), q_codes.data_ptr(), k_codes.data_ptr(), k_codes.stride(0), k_codes.stride(1),
        seq_lens.data_ptr(), _ptr(k_per_seq), k_uniform, k_max, idx.data_ptr(), idx.stride(0), idx.stride(1),
        count.data_ptr(), _ptr(hist_out), _stream(stream)))


def ha_score_topk_per_head(shape: ha_shape, q_codes, k_codes, seq_lens, k_per_seq, k_uniform: int, k_max: int, idx, count,
                           hist_out=None, stream=None) -> None:
    """One list per query head (no group reduction): idx int32 [B,Hq,k_max], count int32 [B,Hq], hist_out [B,Hq,33]."""
    _check("ha_score_topk_per_head", lib().ha_score_topk_per_head(
        C.byref(shape), q_codes.data_ptr(), k_codes.data_ptr(), k_codes.stride(0), k_codes.stride(1),
        seq_lens.data_ptr(), _ptr(k_per_seq), k_uniform, k_max, idx.data_ptr(), idx.stride(0), idx.stride(1),
        count.data_ptr(), _ptr(hist_out), _stream(stream)))


def ha_gather_attn_per_head(shape: ha_shape, q, K, V, seq_lens, idx, count, k_max: int, out, workspace, lse=None,
                            stream=None) -> None:
    """GATHER-ATT through per-query-head lists; workspace sized for the shape with n_kv_heads = n_q_heads."""
    p, n = _ws(workspace)
    kt, vt = make_tensor(K), make_tensor(V)
    _check("ha_gather_attn_per_head", lib().ha_gather_attn_per_head(
        C.byref(shape), q.data_ptr(), C.byref(kt), C.byref(vt), seq_lens.data_ptr(), idx.data_ptr(), idx.stride(0),
        idx.stride(1), count.data_ptr(), k_max, out.data_ptr(), _ptr(lse), p, n, _stream(stream)))


def ha_gather_attn(shape: ha_shape, q, K, V, seq_lens, idx, count, k_max: int, out, workspace, lse=None,
                   stream=None) -> None:
    p, n = _ws(workspace)
    kt, vt = make_tensor(K), make_tensor(V)
    _check("ha_gather_attn", lib().ha_gather_attn(
        C.byref(shape), q.data_ptr(), C.byref(kt), C.byref(vt), seq_lens.data_ptr(), idx.data_ptr(), idx.stride(0),
        idx.stride(1), count.data_ptr(), k_max, out.data_ptr(), _ptr(lse), p, n, _stream(stream)))


def ha_gather_attn_paged(shape: ha_shape, q, K_pool, V_pool, block_table, page_size: int, seq_lens, idx, count, k_max: int,
                         out, workspace, lse=None, stream=None) -> None:
    """K_pool, V_pool: bf16 [n_pages, Hkv, page_size, 128]; block_table: int32 [B, pages per sequence]."""
    p, n = _ws(workspace)
    kt, vt = make_tensor(K_pool), make_tensor(V_pool)
    _check("ha_gather_attn_paged", lib().ha_gather_attn_paged(
        C.byref(shape), q.data_ptr(), C.byref(kt), C.byref(vt), block_table.data_ptr(), block_table.stride(0), page_size,
        seq_lens.data_ptr(), idx.data_ptr(), idx.stride(0), idx.stride(1), count.data_ptr(), k_max, out.data_ptr(),
        _ptr(lse), p, n, _stream(stream)))


def _pool(code_pool: torch.Tensor):
    """int32 [n_pages, Hkv, page_size] signature pool -> (pointer, page stride, head stride, page size)."""
    _dev(code_pool, torch.int32, "code_pool")
    assert code_pool.dim() == 3 and code_pool.stride(2) == 1
    return code_pool.data_ptr(), code_pool.stride(0), code_pool.stride(1), code_pool.shape[2]


def ha_score_topk_paged(shape: ha_shape, q_codes, code_pool, block_table, seq_lens, k_per_seq, k_uniform: int, max_seq_len: int,
                        k_max: int, idx, count, workspace, hist_out=None, per_head: bool = False, stream=None) -> None:
    """ha_score_topk (per_head: ha_score_topk_per_head) over a paged signature pool int32 [n_pages, Hkv, page_size]."""
    p, n = _ws(workspace)
    cp, sp, sh, ps = _pool(code_pool)
    fn = lib().ha_score_topk_per_head_paged if per_head else lib().ha_score_topk_paged
    _check("ha_score_topk_per_head_paged" if per_head else "ha_score_topk_paged", fn(
        C.byref(shape), q_codes.data_ptr(), cp, sp, sh, block_table.data_ptr(), block_table.stride(0), ps, seq_lens.data_ptr(),
        _ptr(k_per_seq), k_uniform, max_seq_len, k_max, idx.data_ptr(), idx.stride(0), idx.stride(1), count.data_ptr(),
        _ptr(hist_out), p, n, _stream(stream)))


def ha_score_topk_per_head_paged(shape: ha_shape, q_codes, code_pool, block_table, seq_lens, k_per_seq, k_uniform: int,
                                 max_seq_len: int, k_max: int, idx, count, workspace, hist_out=None, stream=None) -> None:
    """ha_score_topk_per_head over a paged signature pool; workspace sized for the shape with n_kv_heads = n_q_heads."""
    ha_score_topk_paged(shape, q_codes, code_pool, block_table, seq_lens, k_per_seq, k_uniform, max_seq_len, k_max, idx, count,
                        workspace, hist_out=hist_out, per_head=True, stream=stream)


def ha_gather_attn_per_head_paged(shape: ha_shape, q, K_pool, V_pool, block_table, page_size: int, seq_lens, idx, count,
                                  k_max: int, out, workspace, lse=None, stream=None) -> None:
    p, n = _ws(workspace)
    kt, vt = make_tensor(K_pool), make_tensor(V_pool)
    _check("ha_gather_attn_per_head_paged", lib().ha_gather_attn_per_head_paged(
        C.byref(shape), q.data_ptr(), C.byref(kt), C.byref(vt), block_table.data_ptr(), block_table.stride(0), page_size,
        seq_lens.data_ptr(), idx.data_ptr(), idx.stride(0), idx.stride(1), count.data_ptr(), k_max, out.data_ptr(),
        _ptr(lse), p, n, _stream(stream)))


def ha_encode_append_paged(mapping: Mapping, k_new, code_pool, block_table, seq_lens, stream=None) -> None:
    """Signature of k_new bf16 [B, Hkv, 128] written at token seq_lens[b] - 1 of sequence b in the paged pool."""
    cp, sp, sh, ps = _pool(code_pool)
    _dev(k_new, torch.bfloat16, "k_new")
    assert k_new.is_contiguous()
    _check("ha_encode_append_paged", lib().ha_encode_append_paged(
        mapping.ref, k_new.data_ptr(), k_new.shape[0], cp, sp, sh, block_table.data_ptr(), block_table.stride(0), ps,
        seq_lens.data_ptr(), _stream(stream)))


def ha_sparse_decode_paged_codes(shape: ha_shape, map_q: Mapping, map_k: Optional[Mapping], q, k_new, K_pool, V_pool, code_pool,
                                 block_table, seq_lens, k_per_seq, k_uniform: int, max_seq_len: int, k_max: int, q_codes, idx,
                                 count, out, workspace, lse=None, stream=None) -> None:
    """The whole step with K, V (bf16 [n_pages, Hkv, page_size, 128]) and the signatures (int32 [n_pages, Hkv, page_size])
    all paged through one block table int32 [B, pages]."""
    p, n = _ws(workspace)
    kt, vt = make_tensor(K_pool), make_tensor(V_pool)
    cp, sp, sh, ps = _pool(code_pool)
    _check("ha_sparse_decode_paged_codes", lib().ha_sparse_decode_paged_codes(
        C.byref(shape), map_q.ref, None if map_k is None else map_k.ref, q.data_ptr(), _ptr(k_new), C.byref(kt), C.byref(vt),
        cp, sp, sh, block_table.data_ptr(), block_table.stride(0), ps, seq_lens.data_ptr(), _ptr(k_per_seq), k_uniform,
        max_seq_len, k_max, q_codes.data_ptr(), idx.data_ptr(), idx.stride(0), idx.stride(1), count.data_ptr(), out.data_ptr(),
        _ptr(lse), p, n, _stream(stream)))


def ha_gather_attn_static(shape: ha_shape, q, K, V, seq_lens, idx, count, k_max: int, out, lse=None, stream=None) -> None:
    """ha_gather_attn for callers that cannot allocate a workspace: the scratch is a fixed array inside
    the library (batch * n_kv_heads <= 64).  Make the first call on a device outside stream capture;
    calls that may overlap on the GPU must be ordered by the caller."""
    kt, vt = make_tensor(K), make_tensor(V)
    _check("ha_gather_attn_static", lib().ha_gather_attn_static(
        C.byref(shape), q.data_ptr(), C.byref(kt), C.byref(vt), seq_lens.data_ptr(), idx.data_ptr(), idx.stride(0),
        idx.stride(1), count.data_ptr(), k_max, out.data_ptr(), _ptr(lse), _stream(stream)))


def ha_dense_decode(shape: ha_shape, q, K, V, seq_lens, max_seq_len: int, out, workspace, lse=None,
                    stream=None) -> None:
    p, n = _ws(workspace)
    kt, vt = make_tensor(K), make_tensor(V)
    _check("ha_dense_decode", lib().ha_dense_decode(
        C.byref(shape), q.data_ptr(), C.byref(kt), C.byref(vt), seq_lens.data_ptr(), max_seq_len, out.data_ptr(),
        _ptr(lse), p, n, _stream(stream)))


def ha_sparse_decode(shape: ha_shape, map_q: Mapping, map_k: Optional[Mapping], q, k_new, K, V, k_codes, seq_lens,
                     k_per_seq, k_uniform: int, max_seq_len: int, k_max: int, q_codes, idx, count, out, workspace,
                     lse=None, stream=None) -> None:
    p, n = _ws(workspace)
    kt, vt = make_tensor(K), make_tensor(V)
    _check("ha_sparse_decode", lib().ha_sparse_decode(
        C.byref(shape), map_q.ref, None if map_k is None else map_k.ref, q.data_ptr(), _ptr(k_new), C.byref(kt),
        C.byref(vt), k_codes.data_ptr(), k_codes.stride(0), k_codes.stride(1), seq_lens.data_ptr(), _ptr(k_per_seq),
        k_uniform, max_seq_len, k_max, q_codes.data_ptr(), idx.data_ptr(), idx.stride(0), idx.stride(1),
        count.data_ptr(), out.data_ptr(), _ptr(lse), p, n, _stream(stream)))


def ha_sparse_decode_pipelined(shape: ha_shape, map_q: Mapping, map_k: Optional[Mapping], q, k_new, K, V, k_codes, seq_lens,
                               k_per_seq, k_uniform: int, max_seq_len: int, k_max: int, q_codes, idx, count, out, workspace,
                               lse=None, stream=None) -> None:
    """ha_sparse_decode on the schedule that runs SCORE + TOPK ahead of GATHER-ATT inside one persistent kernel."""
    p, n = _ws(workspace)
    kt, vt = make_tensor(K), make_tensor(V)
    _check("ha_sparse_decode_pipelined", lib().ha_sparse_decode_pipelined(
        C.byref(shape), map_q.ref, None if map_k is None else map_k.ref, q.data_ptr(), _ptr(k_new), C.byref(kt),
        C.byref(vt), k_codes.data_ptr(), k_codes.stride(0), k_codes.stride(1), seq_lens.data_ptr(), _ptr(k_per_seq),
        k_uniform, max_seq_len, k_max, q_codes.data_ptr(), idx.data_ptr(), idx.stride(0), idx.stride(1),
        count.data_ptr(), out.data_ptr(), _ptr(lse), p, n, _stream(stream)))


def ha_sparse_decode_paged(shape: ha_shape, map_q: Mapping, map_k: Optional[Mapping], q, k_new, K_pool, V_pool, block_table,
                           page_size: int, k_codes, seq_lens, k_per_seq, k_uniform: int, max_seq_len: int, k_max: int,
                           q_codes, idx, count, out, workspace, lse=None, stream=None) -> None:
    """The whole step over a paged K/V cache: pools bf16 [n_pages, Hkv, page_size, 128], block_table int32 [B, pages]."""
    p, n = _ws(workspace)
    kt, vt = make_tensor(K_pool), make_tensor(V_pool)
    _check("ha_sparse_decode_paged", lib().ha_sparse_decode_paged(
        C.byref(shape), map_q.ref, None if map_k is None else map_k.ref, q.data_ptr(), _ptr(k_new), C.byref(kt),
        C.byref(vt), block_table.data_ptr(), block_table.stride(0), page_size, k_codes.data_ptr(), k_codes.stride(0),
        k_codes.stride(1), seq_lens.data_ptr(), _ptr(k_per_seq), k_uniform, max_seq_len, k_max, q_codes.data_ptr(),
        idx.data_ptr(), idx.stride(0), idx.stride(1), count.data_ptr(), out.data_ptr(), _ptr(lse), p, n, _stream(stream)))


def ha_sparse_decode_host(shape: ha_shape, map_q: Mapping, map_k: Mapping, q_host, k_new_host, v_new_host, K, V,
                          k_codes, seq_lens, k_per_seq, k_uniform: int, max_seq_len: int, k_max: int, idx, count,
                          out_host, workspace, stream=None) -> None:
    """q_host/k_new_host/v_new_host/out_host: pinned CPU bf16 tensors; everything else on the device."""
    for t in (q_host, k_new_host, v_new_host, out_host):
        if t.is_cuda or not t.is_contiguous():
            raise TypeError("host buffers must be contiguous CPU tensors")
    p, n = _ws(workspace)
    kt, vt = make_tensor(K), make_tensor(V)
    _check("ha_sparse_decode_host", lib().ha_sparse_decode_host(
        C.byref(shape), map_q.ref, map_k.ref, q_host.data_ptr(), k_new_host.data_ptr(), v_new_host.data_ptr(),
        C.byref(kt), C.byref(vt), k_codes.data_ptr(), k_codes.stride(0), k_codes.stride(1), seq_lens.data_ptr(),
        _ptr(k_per_seq), k_uniform, max_seq_len, k_max, idx.data_ptr(), idx.stride(0), idx.stride(1),
        count.data_ptr(), out_host.data_ptr(), p, n, _stream(stream)))


def ha_sparse_decode_paged_host(shape: ha_shape, map_q: Mapping, map_k: Mapping, q_host, k_new_host, v_new_host, K_pool,
                                V_pool, block_table, page_size: int, k_codes, seq_lens, k_per_seq, k_uniform: int,
                                max_seq_len: int, k_max: int, idx, count, out_host, workspace, stream=None) -> None:
    """ha_sparse_decode_host over a paged K/V cache (pools bf16 [n_pages, Hkv, page_size, 128], block_table int32 [B, pages])."""
    for t in (q_host, k_new_host, v_new_host, out_host):
        if t.is_cuda or not t.is_contiguous():
            raise TypeError("host buffers must be contiguous CPU tensors")
    p, n = _ws(workspace)
    kt, vt = make_tensor(K_pool), make_tensor(V_pool)
    _check("ha_sparse_decode_paged_host", lib().ha_sparse_decode_paged_host(
        C.byref(shape), map_q.ref, map_k.ref, q_host.data_ptr(), k_new_host.data_ptr(), v_new_host.data_ptr(),
        C.byref(kt), C.byref(vt), block_table.data_ptr(), block_table.stride(0), page_size, k_codes.data_ptr(),
        k_codes.stride(0), k_codes.stride(1), seq_lens.data_ptr(), _ptr(k_per_seq), k_uniform, max_seq_len, k_max,
        idx.data_ptr(), idx.stride(0), idx.stride(1), count.data_ptr(), out_host.data_ptr(), p, n, _stream(stream)))


class SparseDecodeHostStep:
    """ha_sparse_decode_host with its arguments marshalled once: for a decode loop that reuses the same pinned
    host buffers, device caches and workspace every step, calling the object costs one foreign call instead
    of ~12 us of Python argument handling.  The tensors are kept alive by the object; their addresses, shapes
    and strides must not change (write new q / k_new / v_new values INTO the host buffers)."""

    def __init__(self, shape: ha_shape, map_q: Mapping, map_k: Mapping, q_host, k_new_host, v_new_host, K, V,
                 k_codes, seq_lens, k_per_seq, k_uniform: int, max_seq_len: int, k_max: int, idx, count, out_host,
                 workspace, stream=None):
        for t in (q_host, k_new_host, v_new_host, out_host):
            if t.is_cuda or not t.is_contiguous():
                raise TypeError("host buffers must be contiguous CPU tensors")
        p, n = _ws(workspace)
        self._kt, self._vt = make_tensor(K), make_tensor(V)
        self._keep = (shape, map_q, map_k, q_host, k_new_host, v_new_host, K, V, k_codes, seq_lens, k_per_seq, idx, count,
                      out_host, workspace)
        self._fn = lib().ha_sparse_decode_host
        self._args = (C.byref(shape), map_q.ref, map_k.ref, q_host.data_ptr(), k_new_host.data_ptr(), v_new_host.data_ptr(),
                      C.byref(self._kt), C.byref(self._vt), k_codes.data_ptr(), k_codes.stride(0), k_codes.stride(1),
                      seq_lens.data_ptr(), _ptr(k_per_seq), k_uniform, max_seq_len, k_max, idx.data_ptr(), idx.stride(0),
                      idx.stride(1), count.data_ptr(), out_host.data_ptr(), p, n, _stream(stream))

    def __call__(self) -> None:
        status = self._fn(*self._args)
        if status != HA_OK:
            raise HashAttnError("ha_sparse_decode_host", status)


def ha_read_device_status(workspace, stream=None) -> int:
    flags = C.c_uint32(0)
    _check("ha_read_device_status", lib().ha_read_device_status(workspace.data_ptr(), _stream(stream), C.byref(flags)))
    return int(flags.value)
