"""Small, self-ending run of the decode path for profiler captures (ncu) and quick timing.

    python profile_case.py --config c3 --batch 4 --steps 3

Runs `steps` plain (un-graphed) layer-steps on one replica; inputs are larger than L2 for c3/c4
style shapes but stay within a few GB.  Prints the CUDA-event time per step."""
from __future__ import annotations

import argparse
import dataclasses

import torch

import os
import sys

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2412_14468_b200 import binding as ha  # noqa: E402
from paper_2412_14468_b200 import workloads as wl  # noqa: E402


def prefill(args):
    cfg = wl.CONFIGS[args.config]
    B = args.batch if args.batch is not None else cfg.batch
    T = cfg.n
    assert T is not None, "prefill runs need a config with one fixed length"
    dev = "cuda:0"
    torch.cuda.set_device(0)
    Hkv = cfg.n_kv_heads
    g = torch.Generator(dev).manual_seed(wl.BASE_SEED + 78)
    mp = ha.Mapping(wl.make_mapping(Hkv, g, dev))
    x = torch.randn(B, Hkv, T, 128, device=dev, generator=g).to(torch.bfloat16)
    codes = torch.zeros(B, Hkv, T, dtype=torch.int32, device=dev)
    torch.cuda.synchronize()
    for s in range(args.steps):
        for name, path in (("tcgen05", ha.HA_PREFILL_TCGEN05), ("mma.sync", ha.HA_PREFILL_MMA_SYNC), ("chain-exact fp32", None)):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            if path is None:
                ha.ha_encode(mp, 1, x, codes)             # encode_bulk_kernel: the fma chain of the decode step
            else:
                ha.ha_encode_prefill(mp, 1, x, codes, path=path)
            e1.record()
            torch.cuda.synchronize()
            print(f"step {s} {name}: {e0.elapsed_time(e1) * 1e3:.1f} us")
    print("key bytes per call:", B * Hkv * T * 256, " algorithmic flop per call:", B * Hkv * T * 2 * (128 * 128 * 2 + 128 * 32))


def score_only(args):
    cfg = wl.CONFIGS[args.config]
    B = args.batch if args.batch is not None else cfg.batch
    n, k = cfg.n, cfg.k
    assert n is not None, "score-only runs need a config with one fixed length"
    dev = "cuda:0"
    torch.cuda.set_device(0)
    Hq, Hkv = cfg.n_q_heads, cfg.n_kv_heads
    g = torch.Generator(dev).manual_seed(wl.BASE_SEED + 77)
    kc = torch.randint(-2**31, 2**31 - 1, (B, Hkv, n), dtype=torch.int32, device=dev, generator=g)
    qc = torch.randint(-2**31, 2**31 - 1, (B, Hq), dtype=torch.int32, device=dev, generator=g)
    shape = ha.make_shape(B, Hq, Hkv, 1.0)
    ws = ha.alloc_workspace(shape, n, k, device=dev)
    lens = torch.full((B,), n, dtype=torch.int32, device=dev)
    idx = torch.zeros(B, Hkv, k, dtype=torch.int32, device=dev)
    cnt = torch.zeros(B, Hkv, dtype=torch.int32, device=dev)
    flush = torch.zeros(256 << 20, dtype=torch.uint8, device=dev)
    torch.cuda.synchronize()
    for s in range(args.steps):
        _ = int(flush.sum())
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda._sleep(200000)   # the GPU is busy while the host enqueues: the events bracket the kernels only
        e0.record()
        ha.ha_score_topk(shape, qc, kc, lens, None, k, n, k, idx, cnt, ws)
        e1.record()
        torch.cuda.synchronize()
        print(f"step {s}: {e0.elapsed_time(e1) * 1e3:.1f} us (plain launch, L2 flushed)")
        if args.group_sum:   # the other group reduction: per-head scores added up
            _ = int(flush.sum())
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda._sleep(200000)
            e0.record()
            ha.ha_score_topk_sum(shape, qc, kc, lens, None, k, k, idx, cnt)
            e1.record()
            torch.cuda.synchronize()
            print(f"step {s} summed group scores: {e0.elapsed_time(e1) * 1e3:.1f} us (plain launch, L2 flushed)")
    print("signature bytes per step:", B * Hkv * n * 4)


def score_wide(args):
    """The stand-alone wide-signature SCORE pass and its inner-product comparator on --tokens tokens."""
    dev = "cuda:0"
    torch.cuda.set_device(0)
    n = args.tokens
    g = torch.Generator(dev).manual_seed(wl.BASE_SEED + 5)
    flush = torch.zeros(256 << 20, dtype=torch.uint8, device=dev)
    K = torch.empty(n, 128, device=dev, dtype=torch.bfloat16).normal_(generator=g)
    q = torch.randn(128, device=dev, generator=g).to(torch.bfloat16)
    dots = torch.empty(n, device=dev)
    cases = [("inner product", lambda: ha.ha_inner_products(q, K, dots), n * 260)]
    keep = []
    for bits in (64, 128, 256, 512):
        W = bits // 64
        kc = torch.randint(-2**63, 2**63 - 1, (n, W), dtype=torch.int64, device=dev, generator=g)
        qc = torch.randint(-2**63, 2**63 - 1, (W,), dtype=torch.int64, device=dev, generator=g)
        sc = torch.empty(n, dtype=torch.int16, device=dev)
        keep.append((kc, qc, sc))
        cases.append((f"{bits} bit", (lambda kc=kc, qc=qc, sc=sc, bits=bits: ha.ha_score_wide(qc, kc, bits, sc)), n * (8 * W + 2)))
    torch.cuda.synchronize()
    for s in range(args.steps):
        for name, fn, nbytes in cases:
            _ = int(flush.sum())
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) * 1e3
            print(f"step {s} {name:14s}: {us:9.1f} us  {nbytes / us / 1e3:8.1f} GB/s (plain launch, L2 flushed)")


def encode_only(args):
    """ENCODE of one decode step alone (queries through phi_q, appended keys through phi_kv): a few KB of inputs."""
    cfg = wl.CONFIGS[args.config]
    B = args.batch if args.batch is not None else cfg.batch
    dev = "cuda:0"
    torch.cuda.set_device(0)
    Hq, Hkv = cfg.n_q_heads, cfg.n_kv_heads
    g = torch.Generator(dev).manual_seed(wl.BASE_SEED + 79)
    mq, mk = ha.Mapping(wl.make_mapping(Hkv, g, dev)), ha.Mapping(wl.make_mapping(Hkv, g, dev))
    q = torch.randn(B, Hq, 128, device=dev, generator=g).to(torch.bfloat16)
    k = torch.randn(B, Hkv, 128, device=dev, generator=g).to(torch.bfloat16)
    qc = torch.zeros(B, Hq, 1, dtype=torch.int32, device=dev)
    kc = torch.zeros(B, Hkv, 1, dtype=torch.int32, device=dev)
    flush = torch.zeros(256 << 20, dtype=torch.uint8, device=dev)
    torch.cuda.synchronize()
    for s in range(args.steps):
        _ = int(flush.sum())
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ha.ha_encode(mq, Hq // Hkv, q, qc)
        ha.ha_encode(mk, 1, k, kc)
        e1.record()
        torch.cuda.synchronize()
        print(f"step {s}: {e0.elapsed_time(e1) * 1e3:.1f} us for {B * Hq} + {B * Hkv} vectors (plain launches, L2 flushed)")


def score_topk_wide(args):
    """SCORE + TOPK at signatures of 64 .. 512 bits: one query head over --tokens tokens, k = n / 32."""
    dev = "cuda:0"
    torch.cuda.set_device(0)
    n = args.tokens
    g = torch.Generator(dev).manual_seed(wl.BASE_SEED + 6)
    shape = ha.make_shape(1, 1, 1, 1.0)
    ln = torch.full((1,), n, dtype=torch.int32, device=dev)
    kq = n // 32
    idx = torch.zeros(1, 1, kq, dtype=torch.int32, device=dev)
    cnt = torch.zeros(1, 1, dtype=torch.int32, device=dev)
    ws = ha.alloc_workspace_wide(shape, n, device=dev)
    flush = torch.zeros(256 << 20, dtype=torch.uint8, device=dev)
    cases = []
    for bits in (64, 512):
        W = bits // 64
        kc = torch.randint(-2**63, 2**63 - 1, (1, 1, n, W), dtype=torch.int64, device=dev, generator=g)
        qc = torch.randint(-2**63, 2**63 - 1, (1, 1, W), dtype=torch.int64, device=dev, generator=g)
        cases.append((bits, kc, qc))
    torch.cuda.synchronize()
    for s in range(args.steps):
        for bits, kc, qc in cases:
            _ = int(flush.sum())
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            ha.ha_score_topk_wide(shape, bits, qc, kc, ln, None, kq, n, kq, idx, cnt, ws)
            e1.record()
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) * 1e3
            print(f"step {s} {bits:3d} bit: {us:9.1f} us  {n * bits / 8 / us / 1e3:8.1f} GB/s of signatures (plain launches, L2 flushed)")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="c3")
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--dense", action="store_true", help="also run the dense comparator each step")
    ap.add_argument("--prefill", action="store_true",
                    help="prompt ENCODE alone (tcgen05 and mma.sync kernels) on --batch sequences of the config's length")
    ap.add_argument("--entry-points", action="store_true",
                    help="run the step as its separate entry points (ha_encode, ha_score_topk, ha_gather_attn), i.e. the "
                         "kernels of the three-kernel path, also at batch sizes where ha_sparse_decode is one fused launch")
    ap.add_argument("--wide-index-rows", action="store_true",
                    help="with --entry-points: index rows one entry wider than the budget, which makes ha_gather_attn take "
                         "its split-K kernel also where few units with short rows would get the cluster kernel")
    ap.add_argument("--score-only", action="store_true",
                    help="SCORE + TOPK alone on random signatures (no K/V allocated: large batches stay small)")
    ap.add_argument("--group-sum", action="store_true",
                    help="with --score-only: also run ha_score_topk_sum (per-head scores added instead of maximised)")
    ap.add_argument("--score-wide", action="store_true",
                    help="stand-alone SCORE on signatures of 64..512 bits and the inner-product comparator on --tokens tokens")
    ap.add_argument("--score-topk-wide", action="store_true",
                    help="SCORE + TOPK on signatures of 64 and 512 bits (ha_score_topk_wide) on --tokens tokens")
    ap.add_argument("--encode-only", action="store_true", help="ENCODE of one decode step alone (--batch sequences)")
    ap.add_argument("--pipelined", action="store_true",
                    help="run the step through ha_sparse_decode_pipelined (SCORE + TOPK ahead of GATHER-ATT in one persistent kernel)")
    ap.add_argument("--tokens", type=int, default=1 << 23)
    args = ap.parse_args()
    if args.score_wide:
        return score_wide(args)
    if args.score_topk_wide:
        return score_topk_wide(args)
    if args.encode_only:
        return encode_only(args)
    if args.score_only:
        return score_only(args)
    if args.prefill:
        return prefill(args)
    cfg = wl.CONFIGS[args.config]
    if args.batch is not None:
        cfg = dataclasses.replace(cfg, batch=args.batch)
    dev = "cuda:0"
    torch.cuda.set_device(0)
    w = wl.make_workload(cfg, dev)
    B, Hq, Hkv = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads
    shape = ha.make_shape(B, Hq, Hkv, w["sm_scale"])
    ws = ha.alloc_workspace(shape, w["n_cap"], w["k_max"], device=dev)
    mq, mk = ha.Mapping(w["map_q"]), ha.Mapping(w["map_k"])
    kc = torch.zeros(B, Hkv, (w["n_cap"] + 3) // 4 * 4, dtype=torch.int32, device=dev)
    ha.ha_encode(mk, 1, w["K"], kc)
    qc = torch.zeros(B, Hq, dtype=torch.int32, device=dev)
    row_width = w["k_max"] + (2049 - w["k_max"] if args.wide_index_rows and w["k_max"] <= 2048 else 0)
    idx = torch.zeros(B, Hkv, row_width, dtype=torch.int32, device=dev)
    cnt = torch.zeros(B, Hkv, dtype=torch.int32, device=dev)
    out = torch.zeros(B, Hq, 128, dtype=torch.bfloat16, device=dev)
    flush = torch.zeros(256 << 20, dtype=torch.uint8, device=dev)
    last_slot = (w["seq_lens"] - 1).to(torch.int32)   # where the appended key's signature goes
    torch.cuda.synchronize()
    for s in range(args.steps):
        _ = int(flush.sum())                       # read 256 MB: evicts L2 and leaves only clean lines
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        if args.entry_points:
            ha.ha_encode(mq, Hq // Hkv, w["q"], qc.view(B, Hq, 1))
            ha.ha_encode(mk, 1, w["k_new"], kc, slot=last_slot)
            ha.ha_score_topk(shape, qc, kc, w["seq_lens"], w["k_per_seq"], 0, w["n_cap"], w["k_max"], idx, cnt, ws)
            ha.ha_gather_attn(shape, w["q"], w["K"], w["V"], w["seq_lens"], idx, cnt, row_width, out, ws)
        else:
            step = ha.ha_sparse_decode_pipelined if args.pipelined else ha.ha_sparse_decode
            step(shape, mq, mk, w["q"], w["k_new"], w["K"], w["V"], kc, w["seq_lens"], w["k_per_seq"], 0,
                 w["n_cap"], w["k_max"], qc, idx, cnt, out, ws)
        e1.record()
        if args.dense:
            ha.ha_dense_decode(shape, w["q"], w["K"], w["V"], w["seq_lens"], w["n_cap"], out, ws)
        torch.cuda.synchronize()
        print(f"step {s}: {e0.elapsed_time(e1) * 1e3:.1f} us (plain launches, L2 flushed)")
    assert ha.ha_read_device_status(ws) == 0
    print("algorithmic bytes per step:", wl.algorithmic_bytes(w["lens"], w["ks"], Hq, Hkv))


if __name__ == "__main__":
    main()
