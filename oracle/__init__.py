"""ctypes front end of the C oracle (oracle/ha_oracle.c).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg import this package; the CUDA
library and its Python binding never do.  bf16 data travels as numpy uint16 arrays holding the
raw bit patterns.
"""
from __future__ import annotations

import ctypes as C
import math

import numpy as np

from .build import build as _build

_lib = None

D = 128
HID = 128
BITS = 32


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build())
        _lib.ora_topk.restype = C.c_int64
        _lib.ora_topk_windows.restype = C.c_int64
        _lib.ora_f64_to_bf16.restype = C.c_uint16
        _lib.ora_f64_to_bf16.argtypes = [C.c_double]
        _lib.ora_max_threads.restype = C.c_int32
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def bf16_bits_to_f64(a) -> np.ndarray:
    """Exact value of bf16 bit patterns, as float64."""
    a = np.ascontiguousarray(a, dtype=np.uint16)
    return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f64_to_bf16_bits(x: float) -> int:
    return int(lib().ora_f64_to_bf16(float(x)))


def encode(x, w1, w2, w3, b1=None, b2=None, b3=None, return_z3=False):
    """Eq. 2 for one mapping.  x: uint16 [n,128]; w1,w2: uint16 [128,128]; w3: uint16 [128,32]."""
    x = _u16(x).reshape(-1, D)
    n = x.shape[0]
    w1, w2, w3 = _u16(w1), _u16(w2), _u16(w3)
    assert w1.shape == (D, HID) and w2.shape == (HID, HID) and w3.shape == (HID, BITS)
    bs = [None if b is None else np.ascontiguousarray(b, dtype=np.float32) for b in (b1, b2, b3)]
    codes = np.zeros(n, dtype=np.uint32)
    z3 = np.zeros((n, BITS), dtype=np.float32) if return_z3 else None
    lib().ora_encode(_p(x), C.c_int64(n), C.c_int64(D), _p(w1), _p(w2), _p(w3),
                     _p(bs[0]), _p(bs[1]), _p(bs[2]), _p(codes), _p(z3))
    return (codes, z3) if return_z3 else codes


def encode_wide(x, w1, w2, w3, b1=None, b2=None, b3=None, return_z3=False):
    """Eq. 2 at b = w3.shape[1] bits (a multiple of 64).  x: uint16 [n,128]; w3: uint16 [128,b]; codes uint64 [n, b/64]
    with bit j of a signature = bit j % 64 of word j // 64."""
    x = _u16(x).reshape(-1, D)
    n = x.shape[0]
    w1, w2, w3 = _u16(w1), _u16(w2), _u16(w3)
    n_bits = w3.shape[1]
    assert w1.shape == (D, HID) and w2.shape == (HID, HID) and w3.shape == (HID, n_bits) and n_bits % 64 == 0
    bs = [None if b is None else np.ascontiguousarray(b, dtype=np.float32) for b in (b1, b2, b3)]
    codes = np.zeros((n, n_bits // 64), dtype=np.uint64)
    z3 = np.zeros((n, n_bits), dtype=np.float32) if return_z3 else None
    lib().ora_encode_wide(_p(x), C.c_int64(n), C.c_int64(D), _p(w1), _p(w2), _p(w3), _p(bs[0]), _p(bs[1]), _p(bs[2]),
                          C.c_int32(n_bits), _p(codes), _p(z3))
    return (codes, z3) if return_z3 else codes


def score_wide_group(qcodes, kcodes) -> np.ndarray:
    """Group score at b bits: the maximum over the group's query signatures (qcodes uint64 [G, W]) of the pinned
    single-query score_wide, as the 32-bit layer-step reduces a GQA group; kcodes uint64 [n, W]."""
    qcodes = np.ascontiguousarray(qcodes, dtype=np.uint64)
    best = score_wide(qcodes[0], kcodes)
    for j in range(1, qcodes.shape[0]):
        best = np.maximum(best, score_wide(qcodes[j], kcodes))
    return best


def score(qcodes, kcodes) -> np.ndarray:
    """Eq. 1 as 32 - Hamming, maximum over the query codes of one GQA group."""
    qcodes = np.ascontiguousarray(qcodes, dtype=np.uint32).reshape(-1)
    kcodes = np.ascontiguousarray(kcodes, dtype=np.uint32).reshape(-1)
    out = np.zeros(kcodes.shape[0], dtype=np.int32)
    lib().ora_score(_p(qcodes), C.c_int32(qcodes.shape[0]), _p(kcodes), C.c_int64(kcodes.shape[0]), _p(out))
    return out


def score_sum(qcodes, kcodes) -> np.ndarray:
    """Eq. 1 per query code, summed over the query codes of one GQA group (range 0 .. 32 * group)."""
    qcodes = np.ascontiguousarray(qcodes, dtype=np.uint32).reshape(-1)
    kcodes = np.ascontiguousarray(kcodes, dtype=np.uint32).reshape(-1)
    out = np.zeros(kcodes.shape[0], dtype=np.int32)
    lib().ora_score_sum(_p(qcodes), C.c_int32(qcodes.shape[0]), _p(kcodes), C.c_int64(kcodes.shape[0]), _p(out))
    return out


def score_wide(qcode, kcodes) -> np.ndarray:
    """Score of the SCORE-latency table: b - Hamming for signatures of b = 64 * W bits, kcodes uint64 [n, W]."""
    qcode = np.ascontiguousarray(qcode, dtype=np.uint64).reshape(-1)
    kcodes = np.ascontiguousarray(kcodes, dtype=np.uint64)
    assert kcodes.ndim == 2 and kcodes.shape[1] == qcode.shape[0]
    out = np.zeros(kcodes.shape[0], dtype=np.int32)
    lib().ora_score_wide(_p(qcode), _p(kcodes), C.c_int64(kcodes.shape[0]), C.c_int32(qcode.shape[0]), _p(out))
    return out


def inner_products(q, K) -> np.ndarray:
    """<q, K_i> for bf16 bit patterns q [128], K [n, 128]; float64 accumulation."""
    q = _u16(q).reshape(-1)
    K = _u16(K)
    assert q.shape[0] == D and K.ndim == 2 and K.shape[1] == D
    out = np.zeros(K.shape[0], dtype=np.float64)
    lib().ora_inner_products(_p(q), _p(K), C.c_int64(K.shape[0]), C.c_int64(D), _p(out))
    return out


def topk(scores, k: int) -> np.ndarray:
    """Standard top-k with ties to the lowest token index; indices returned ascending."""
    scores = np.ascontiguousarray(scores, dtype=np.int32).reshape(-1)
    n = scores.shape[0]
    out = np.full(max(min(k, n), 1), -1, dtype=np.int32)
    cnt = lib().ora_topk(_p(scores), C.c_int64(n), C.c_int64(k), _p(out))
    return out[:cnt].copy()


def topk_windows(scores, k: int, n_sink: int, n_local: int) -> np.ndarray:
    """The first n_sink and the last n_local tokens always, plus the top k of the others (Section 5,
    paragraph on baselines); indices returned ascending."""
    scores = np.ascontiguousarray(scores, dtype=np.int32).reshape(-1)
    n = scores.shape[0]
    out = np.full(max(n, 1), -1, dtype=np.int32)
    cnt = lib().ora_topk_windows(_p(scores), C.c_int64(n), C.c_int64(k), C.c_int64(n_sink), C.c_int64(n_local), _p(out))
    return out[:cnt].copy()


def gather_attn(q, K, V, idx, sm_scale=None, n_valid=None):
    """GATHER-ATT for one query head.  q: uint16 [128]; K, V: uint16 [n,128]; idx: int32 list or None.
    Returns (out uint16 [128], lse float, out float64 [128])."""
    q = _u16(q).reshape(D)
    K, V = _u16(K).reshape(-1, D), _u16(V).reshape(-1, D)
    n = K.shape[0]
    if sm_scale is None:
        sm_scale = 1.0 / math.sqrt(D)
    if n_valid is None:
        n_valid = n
    if idx is None:
        ip, count = None, n_valid
    else:
        idx = np.ascontiguousarray(idx, dtype=np.int32).reshape(-1)
        ip, count = _p(idx), idx.shape[0]
    out = np.zeros(D, dtype=np.uint16)
    out64 = np.zeros(D, dtype=np.float64)
    lse = C.c_double(0.0)
    lib().ora_gather_attn(_p(q), _p(K), _p(V), C.c_int64(D), ip, C.c_int64(count), C.c_int64(n_valid),
                          C.c_double(sm_scale), _p(out), C.byref(lse), _p(out64))
    return out, lse.value, out64


def unpage_rows(pool, block_table_row, page_size: int, head: int, n: int) -> np.ndarray:
    """Rows 0..n-1 of one sequence and KV head out of a paged cache (Section 4.4: K/V are read in place; the
    vLLM integration keeps them in pages): pool is [n_pages, Hkv, page_size, 128]; token t lives in page
    block_table_row[t // page_size] at slot t % page_size.  Paging is storage only: GATHER-ATT over a paged
    cache is gather_attn over these rows."""
    pool = _u16(pool)
    t = np.arange(n)
    pages = np.asarray(block_table_row, dtype=np.int64)[t // page_size]
    return np.ascontiguousarray(pool[pages, head, t % page_size, :])


def unpage_codes(pool, block_table_row, page_size: int, head: int, n: int) -> np.ndarray:
    """Signatures 0..n-1 of one sequence and KV head out of a paged signature cache: pool is uint32 [n_pages, Hkv,
    page_size]; token t lives in page block_table_row[t // page_size] at slot t % page_size.  Paging is storage only:
    SCORE + TOPK over a paged cache is score / topk over these signatures."""
    pool = np.ascontiguousarray(pool, dtype=np.uint32)
    t = np.arange(n)
    pages = np.asarray(block_table_row, dtype=np.int64)[t // page_size]
    return np.ascontiguousarray(pool[pages, head, t % page_size])


def dense(q, K, V, n=None, sm_scale=None):
    """SDPA for one query over tokens 0..n-1."""
    return gather_attn(q, K, V, None, sm_scale=sm_scale, n_valid=n)


def max_threads() -> int:
    return int(lib().ora_max_threads())


def decode_step(q, k_new, K, V, kcodes, map_q, map_k, seq_lens, k_per_seq, sm_scale=None, n_threads=1,
                n_sink=0, n_local=0):
    """One layer-step: ENCODE -> SCORE -> TOPK -> GATHER-ATT for the batch.

    q uint16 [B,Hq,128]; k_new uint16 [B,Hkv,128] or None; K, V uint16 [B,Hkv,n_cap,128];
    kcodes uint32 [B,Hkv,n_cap] (slot n_b-1 is overwritten when k_new is given);
    map_q / map_k: dict with w1,w2,w3 (uint16 [Hkv,...]) and b1,b2,b3 (float32 [Hkv,out] or None).
    n_sink / n_local: tokens always kept in addition to the budget (0, 0 = plain top-k).
    Returns dict(qcodes, idx, count, out, lse)."""
    q = _u16(q)
    B, Hq, _ = q.shape
    K, V = _u16(K), _u16(V)
    Hkv, n_cap = K.shape[1], K.shape[2]
    assert kcodes.dtype == np.uint32 and kcodes.flags.c_contiguous and kcodes.shape == (B, Hkv, n_cap)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    k_per_seq = np.ascontiguousarray(k_per_seq, dtype=np.int32)
    k_max = max(int(k_per_seq.max()) + int(n_sink) + int(n_local), 1)
    if sm_scale is None:
        sm_scale = 1.0 / math.sqrt(D)

    def m(mp):
        ws = [_u16(mp[k]) for k in ("w1", "w2", "w3")]
        bs = [None if mp.get(k) is None else np.ascontiguousarray(mp[k], dtype=np.float32)
              for k in ("b1", "b2", "b3")]
        return ws, bs

    (wq, bq), (wk, bk) = m(map_q), m(map_k)
    k_new = None if k_new is None else _u16(k_new)
    qcodes = np.zeros((B, Hq), dtype=np.uint32)
    idx = np.full((B, Hkv, k_max), -1, dtype=np.int32)
    count = np.zeros((B, Hkv), dtype=np.int32)
    out = np.zeros((B, Hq, D), dtype=np.uint16)
    lse = np.zeros((B, Hq), dtype=np.float64)
    lib().ora_decode_step(
        C.c_int32(B), C.c_int32(Hq), C.c_int32(Hkv), C.c_int64(n_cap), C.c_int64(k_max),
        _p(q), _p(k_new), _p(K), _p(V), _p(kcodes),
        _p(wq[0]), _p(wq[1]), _p(wq[2]), _p(bq[0]), _p(bq[1]), _p(bq[2]),
        _p(wk[0]), _p(wk[1]), _p(wk[2]), _p(bk[0]), _p(bk[1]), _p(bk[2]),
        _p(seq_lens), _p(k_per_seq), C.c_double(sm_scale),
        _p(qcodes), _p(idx), _p(count), _p(out), _p(lse), C.c_int32(n_threads), C.c_int32(n_sink), C.c_int32(n_local))
    return dict(qcodes=qcodes, idx=idx, count=count, out=out, lse=lse)
