"""Seeded synthetic decode workloads (inputs only; none of the method's arithmetic lives here).

The tensors stand in for Llama-3.1-8B-Instruct decode shapes (32 query heads, 8 KV heads,
head_dim 128; Section 5 "Models and datasets") on long-context prompts: the paper's data and
weights are not available, so q, K, V are unit normals rounded to bf16, with a fraction of
"pivotal" keys planted as scaled copies of a query direction (Section 1 calls the few tokens
that dominate the softmax pivotal).  The mapping networks are random-init (uniform within
+-1/sqrt(fan_in)) with the shapes of Section 5.2.  The generator serves the CUDA path, the
tests and the CPU oracle alike; it produces data, never codes, scores or outputs.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Sequence, Union

import torch

D = 128
HID = 128
BITS = 32
BASE_SEED = 241214468


@dataclasses.dataclass(frozen=True)
class Config:
    name: str
    index: int                       # offset added to BASE_SEED
    batch: int
    n: Union[int, Sequence[int], None]   # context length per sequence; None = ragged draw
    k: Optional[int]                 # budget; None = n_b // sparsity
    planted: float                   # fraction of keys planted per (b, KV head)
    n_q_heads: int = 32
    n_kv_heads: int = 8
    sparsity: int = 32
    n_lo: int = 8192                 # ragged draw bounds (inclusive)
    n_hi: int = 131072


CONFIGS: Dict[str, Config] = {
    "c1": Config("c1", 0, 1, 4096, 256, 0.0, sparsity=16),
    "c2": Config("c2", 1, 1, 32768, 1024, 0.01, sparsity=32),
    "c3": Config("c3", 2, 16, 32768, 2048, 0.01, sparsity=16),
    "c4": Config("c4", 3, 1, 524288, 16384, 0.001, sparsity=32),
    "c5": Config("c5", 4, 32, None, None, 0.01, sparsity=32),
}


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _bf16_normal(shape, gen, device, chunk_rows: int = 1 << 22) -> torch.Tensor:
    """randn in fp32 rounded to bf16, produced in chunks so that the fp32 transient stays small."""
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    flat = out.view(-1)
    total = flat.numel()
    step = chunk_rows * 16
    for s in range(0, total, step):
        e = min(total, s + step)
        flat[s:e] = torch.randn(e - s, generator=gen, device=device, dtype=torch.float32).to(torch.bfloat16)
    return out


def _uniform(shape, bound: float, gen, device, dtype) -> torch.Tensor:
    u = torch.rand(shape, generator=gen, device=device, dtype=torch.float32)
    return ((u * 2.0 - 1.0) * bound).to(dtype)


def make_mapping(n_kv_heads: int, gen, device) -> Dict[str, torch.Tensor]:
    """One mapping network per KV head: W1,W2 [Hkv,128,128], W3 [Hkv,128,32] bf16 ([in][out]),
    biases fp32."""
    b = 1.0 / math.sqrt(D)
    return {
        "w1": _uniform((n_kv_heads, D, HID), b, gen, device, torch.bfloat16),
        "b1": _uniform((n_kv_heads, HID), b, gen, device, torch.float32),
        "w2": _uniform((n_kv_heads, HID, HID), b, gen, device, torch.bfloat16),
        "b2": _uniform((n_kv_heads, HID), b, gen, device, torch.float32),
        "w3": _uniform((n_kv_heads, HID, BITS), b, gen, device, torch.bfloat16),
        "b3": _uniform((n_kv_heads, BITS), b, gen, device, torch.float32),
    }


def make_workload(cfg: Union[str, Config], device: Union[str, torch.device] = "cpu",
                  seed: Optional[int] = None) -> Dict[str, object]:
    """Build one layer's decode inputs.

    Returns a dict with
      q [B,Hq,128] bf16, K,V [B,Hkv,n_cap,128] bf16 (slots >= n_b are zero and never read),
      k_new [B,Hkv,128] bf16 (= K[:, :, n_b-1], the key appended this step),
      map_q, map_k (dicts of weights), seq_lens [B] int32, k_per_seq [B] int32,
      n_cap, k_max, cfg.
    Generators are seeded BASE_SEED + cfg.index (+ 1000 * position in the order
    q, K, V, weights, planted positions, lengths)."""
    if isinstance(cfg, str):
        cfg = CONFIGS[cfg]
    device = torch.device(device)
    base = (BASE_SEED + cfg.index) if seed is None else seed
    B, Hq, Hkv = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads
    G = Hq // Hkv

    # lengths first (they fix the shapes) but from their own generator (last in the seed order)
    if cfg.n is None:
        lens = torch.randint(cfg.n_lo, cfg.n_hi + 1, (B,), generator=_gen("cpu", base + 5000)).tolist()
    elif isinstance(cfg.n, int):
        lens = [cfg.n] * B
    else:
        lens = list(cfg.n)
        assert len(lens) == B
    ks = [(n // cfg.sparsity) if cfg.k is None else cfg.k for n in lens]
    n_cap = max(max(lens), 1)
    k_max = max(max(ks), 1)

    q = _bf16_normal((B, Hq, D), _gen(device, base + 0), device)
    K = _bf16_normal((B, Hkv, n_cap, D), _gen(device, base + 1000), device)
    V = _bf16_normal((B, Hkv, n_cap, D), _gen(device, base + 2000), device)
    gw = _gen(device, base + 3000)
    map_q = make_mapping(Hkv, gw, device)
    map_k = make_mapping(Hkv, gw, device)

    # planted pivotal keys: scaled copies (x4 after normalisation) of the group's query directions
    gp = _gen(device, base + 4000)
    qf = q.to(torch.float32)
    qdir = 4.0 * qf / qf.norm(dim=-1, keepdim=True).clamp_min(1e-20)
    planted: List[List[torch.Tensor]] = []
    for b in range(B):
        row = []
        for g in range(Hkv):
            m = int(math.floor(cfg.planted * lens[b]))
            if m > 0:
                pos = torch.randperm(lens[b], generator=gp, device=device)[:m]
                heads = g * G + (torch.arange(m, device=device) % G)
                K[b, g, pos] = qdir[b, heads].to(torch.bfloat16)
            else:
                pos = torch.empty(0, dtype=torch.int64, device=device)
            row.append(pos)
        planted.append(row)
        if lens[b] < n_cap:
            K[b, :, lens[b]:] = 0
            V[b, :, lens[b]:] = 0

    last = torch.tensor([max(n - 1, 0) for n in lens], device=device)
    k_new = K[torch.arange(B, device=device), :, last].contiguous()        # [B,Hkv,128]
    v_new = V[torch.arange(B, device=device), :, last].contiguous()
    return {
        "cfg": cfg, "q": q, "K": K, "V": V, "k_new": k_new, "v_new": v_new,
        "map_q": map_q, "map_k": map_k,
        "seq_lens": torch.tensor(lens, dtype=torch.int32, device=device),
        "k_per_seq": torch.tensor(ks, dtype=torch.int32, device=device),
        "lens": lens, "ks": ks, "n_cap": n_cap, "k_max": k_max, "planted": planted,
        "sm_scale": 1.0 / math.sqrt(D),
    }


def shard_heads(w: Dict[str, object], rank: int, world: int) -> Dict[str, object]:
    """Head-parallel split of one layer's inputs: rank r of `world` keeps KV heads [r * Hkv / world, (r + 1) * Hkv /
    world), their query heads and their mapping networks; lengths and budgets are shared.  The (sequence, KV head)
    units of the path are independent, so the shards need no exchange: every rank runs the whole step on its heads and
    the outputs are the corresponding slices of the unsharded result.  K and V come back as strided views (the entry
    points take strides), everything else contiguous."""
    cfg = w["cfg"]
    Hq, Hkv = cfg.n_q_heads, cfg.n_kv_heads
    assert 0 <= rank < world and Hkv % world == 0, "the KV heads must divide evenly over the ranks"
    hk, G = Hkv // world, Hq // Hkv
    kv = slice(rank * hk, (rank + 1) * hk)
    qh = slice(rank * hk * G, (rank + 1) * hk * G)
    out = dict(w)
    out["cfg"] = dataclasses.replace(cfg, n_q_heads=hk * G, n_kv_heads=hk)
    out["q"] = w["q"][:, qh].contiguous()
    out["K"], out["V"] = w["K"][:, kv], w["V"][:, kv]
    out["k_new"], out["v_new"] = w["k_new"][:, kv].contiguous(), w["v_new"][:, kv].contiguous()
    out["map_q"] = {k: v[kv].contiguous() for k, v in w["map_q"].items()}
    out["map_k"] = {k: v[kv].contiguous() for k, v in w["map_k"].items()}
    out["planted"] = [row[kv] for row in w["planted"]]
    return out


def algorithmic_bytes(lens: Sequence[int], ks: Sequence[int], n_q_heads: int = 32, n_kv_heads: int = 8) -> int:
    """Bytes one sparse layer-step must move: 4 B of key code per cached token, 512 B of K and V
    rows per selected token (per KV head), 512 B of q and out per query head."""
    total = 0
    for n, k in zip(lens, ks):
        total += n_kv_heads * (4 * n + 512 * min(k, n)) + n_q_heads * 512
    return total


def dense_bytes(lens: Sequence[int], n_q_heads: int = 32, n_kv_heads: int = 8) -> int:
    return sum(n_kv_heads * 512 * n + n_q_heads * 512 for n in lens)


def as_u16(t: torch.Tensor):
    """bf16 tensor -> numpy uint16 bit patterns (host copy)."""
    return t.detach().to("cpu").contiguous().view(torch.int16).numpy().view("uint16")


def mapping_numpy(mp: Dict[str, torch.Tensor]) -> Dict[str, object]:
    out = {}
    for k, v in mp.items():
        out[k] = as_u16(v) if v.dtype == torch.bfloat16 else v.detach().to("cpu").contiguous().numpy()
    return out
