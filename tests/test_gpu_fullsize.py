"""GPU parity at the benchmark's full sizes (configs c2..c5), through the same entry point and
launch configuration that bench.py times (ha_sparse_decode on device-resident inputs).

What the oracle can recompute in seconds is checked exhaustively (query codes, scores via the
histogram, counts and index sets of every (sequence, KV head) unit, against the oracle run on the
same signature cache); the signature cache itself and the attention outputs are checked on samples
(tokens / heads drawn from a seeded generator), each sample computed by the oracle one by one."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2412_14468_b200 import binding as ha
from paper_2412_14468_b200 import workloads as wl
from tests._util import OUT_TOL, assert_out_close, codes_np, max_abs_diff_bf16, u16

pytestmark = pytest.mark.gpu
DEV = "cuda"


# the bench's batch sweep at the headline shape: one fused launch with clusters of 8 (32 units) and of 4 (64 units)
SWEEP = {f"sweep_B{bsz}_32K_32x": wl.Config(f"sweep{bsz}", 10 + bsz, bsz, 32768, 1024, 0.01) for bsz in (4, 8)}


def _run(cfg_name, n_sink=0, n_local=0):
    w = wl.make_workload(SWEEP.get(cfg_name, cfg_name), DEV)
    if n_sink or n_local:
        w = dict(w, k_max=w["k_max"] + n_sink + n_local)      # the index rows hold the always-kept tokens too
    cfg = w["cfg"]
    B, Hq, Hkv = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads
    shape = ha.make_shape(B, Hq, Hkv, w["sm_scale"], n_sink=n_sink, n_local=n_local)
    ws = ha.alloc_workspace(shape, w["n_cap"], w["k_max"])
    mq, mk = ha.Mapping(w["map_q"]), ha.Mapping(w["map_k"])
    kc = torch.zeros(B, Hkv, (w["n_cap"] + 3) // 4 * 4, dtype=torch.int32, device=DEV)
    ha.ha_encode(mk, 1, w["K"], kc)
    for b in range(B):
        kc[b, :, w["lens"][b] - 1] = 0x13572468           # stale value in the appended slot
    qc = torch.zeros(B, Hq, dtype=torch.int32, device=DEV)
    idx = torch.zeros(B, Hkv, w["k_max"], dtype=torch.int32, device=DEV)
    cnt = torch.zeros(B, Hkv, dtype=torch.int32, device=DEV)
    out = torch.zeros(B, Hq, 128, dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros(B, Hq, device=DEV)
    for _ in range(2):                                      # twice: the workspace must be reusable as is
        ha.ha_sparse_decode(shape, mq, mk, w["q"], w["k_new"], w["K"], w["V"], kc, w["seq_lens"], w["k_per_seq"], 0,
                            w["n_cap"], w["k_max"], qc, idx, cnt, out, ws, lse=lse)
    torch.cuda.synchronize()
    assert ha.ha_read_device_status(ws) == 0
    hist = torch.zeros(B, Hkv, 33, dtype=torch.int32, device=DEV)
    idx2, cnt2 = torch.zeros_like(idx), torch.zeros_like(cnt)
    ha.ha_score_topk(shape, qc, kc, w["seq_lens"], w["k_per_seq"], 0, w["n_cap"], w["k_max"], idx2, cnt2, ws, hist_out=hist)
    assert torch.equal(idx2, idx) and torch.equal(cnt2, cnt)
    return w, dict(kc=kc, qc=qc, idx=idx, cnt=cnt, out=out, lse=lse, hist=hist, shape=shape, ws=ws)


@pytest.mark.parametrize("cfg_name", ["c2", "c3", "c4", "c5", "sweep_B4_32K_32x", "sweep_B8_32K_32x", "c2+sink128+local128"])
def test_full_size_config_matches_oracle(cfg_name):
    import time
    t_start = time.time()
    n_sink, n_local = (128, 128) if cfg_name.endswith("+sink128+local128") else (0, 0)   # the bench's window line
    cfg_name = cfg_name.split("+")[0]
    w, r = _run(cfg_name, n_sink, n_local)
    t_gpu = time.time() - t_start
    cfg = w["cfg"]
    B, Hq, Hkv = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads
    G = Hq // Hkv
    rng = np.random.default_rng(2412 + cfg.index)
    mq, mk = wl.mapping_numpy(w["map_q"]), wl.mapping_numpy(w["map_k"])
    qu = u16(w["q"])
    kc_np = codes_np(r["kc"])
    qc_np = codes_np(r["qc"])
    idx_np, cnt_np, hist_np = r["idx"].cpu().numpy(), r["cnt"].cpu().numpy(), r["hist"].cpu().numpy()
    ou = u16(r["out"])
    lse_np = r["lse"].cpu().numpy()

    # ---- query signatures: all, bit for bit
    for b in range(B):
        for g in range(Hkv):
            exp = oracle.encode(qu[b, g * G:(g + 1) * G], mq["w1"][g], mq["w2"][g], mq["w3"][g], mq["b1"][g], mq["b2"][g], mq["b3"][g])
            assert np.array_equal(qc_np[b, g * G:(g + 1) * G], exp)

    # ---- SCORE + TOPK on the same signature cache: every unit, bit for bit (stage isolation)
    for b in range(B):
        n, k = w["lens"][b], w["ks"][b]
        for g in range(Hkv):
            s = oracle.score(qc_np[b, g * G:(g + 1) * G], kc_np[b, g, :n])
            counted = s[n_sink:max(n - n_local, n_sink)]               # always-kept tokens are not counted
            assert np.array_equal(hist_np[b, g], np.bincount(counted, minlength=33)), (b, g)
            exp = oracle.topk_windows(s, k, n_sink, n_local) if (n_sink or n_local) else oracle.topk(s, k)
            assert cnt_np[b, g] == len(exp)
            if not (n_sink or n_local):
                assert len(exp) == min(k, n)
            assert np.array_equal(idx_np[b, g, :len(exp)], exp), (b, g)
            assert np.all(idx_np[b, g, len(exp):] == -1)

    # ---- signature cache: sampled tokens (the appended slot, planted keys, selected tokens, random ones)
    units = [(b, g) for b in range(B) for g in range(Hkv)]
    for (b, g) in [units[i] for i in rng.choice(len(units), size=min(8, len(units)), replace=False)]:
        n = w["lens"][b]
        pos = np.unique(np.concatenate([
            [n - 1, 0], w["planted"][b][g].cpu().numpy()[:256], idx_np[b, g, :min(cnt_np[b, g], 1024)],
            rng.integers(0, n, size=2048)])).astype(np.int64)
        rows = u16(w["K"][b, g, torch.from_numpy(pos).to(DEV)])
        exp = oracle.encode(rows, mk["w1"][g], mk["w2"][g], mk["w3"][g], mk["b1"][g], mk["b2"][g], mk["b3"][g])
        assert np.array_equal(kc_np[b, g, pos], exp), (b, g)

    # ---- GATHER-ATT: sampled query heads, each recomputed by the oracle from the selected rows
    heads = [(b, h) for b in range(B) for h in range(Hq)]
    worst = 0.0
    for (b, h) in [heads[i] for i in rng.choice(len(heads), size=min(24, len(heads)), replace=False)]:
        g = h // G
        sel = torch.from_numpy(idx_np[b, g, :cnt_np[b, g]].astype(np.int64)).to(DEV)
        Kr, Vr = u16(w["K"][b, g, sel]), u16(w["V"][b, g, sel])
        eo, el, _ = oracle.gather_attn(qu[b, h], Kr, Vr, None, sm_scale=w["sm_scale"])
        worst = max(worst, max_abs_diff_bf16(ou[b, h], eo))
        assert abs(lse_np[b, h] - el) < 1e-3 * max(1.0, abs(el))
    assert worst <= OUT_TOL, worst

    # ---- properties that hold at any size: ascending indices inside the sequence, finite outputs
    for b in range(B):
        for g in range(Hkv):
            sel = idx_np[b, g, :cnt_np[b, g]]
            assert np.all(np.diff(sel) > 0) and (len(sel) == 0 or (sel[0] >= 0 and sel[-1] < w["lens"][b]))
    assert np.isfinite(oracle.bf16_bits_to_f64(ou)).all()

    print(f"{cfg_name}: lens[:4]={w['lens'][:4]} ks[:4]={w['ks'][:4]} tokens scored by the oracle="
          f"{sum(w['lens']) * Hkv}, gpu+generation {t_gpu:.1f}s, total {time.time() - t_start:.1f}s, worst |out diff| {worst:.2e}")
    if cfg_name == "c2":
        # dense comparator at full context against the oracle on sampled heads
        dense = torch.zeros_like(r["out"])
        ha.ha_dense_decode(r["shape"], w["q"], w["K"], w["V"], w["seq_lens"], w["n_cap"], dense, r["ws"])
        Ku, Vu = u16(w["K"]), u16(w["V"])
        for h in (0, 13, 31):
            eo, _, _ = oracle.dense(qu[0, h], Ku[0, h // G], Vu[0, h // G], n=w["lens"][0], sm_scale=w["sm_scale"])
            assert max_abs_diff_bf16(u16(dense)[0, h], eo) <= OUT_TOL


@pytest.mark.parametrize("B", [130, 74, 50])
def test_many_units(B):
    # 130 sequences: more than 1024 (sequence, KV head) units, the attention kernel maps one CTA to each unit;
    # 74: twice as many units as CTA slots, whole units per CTA; 50: more units than CTAs, units split over CTAs
    cfg = wl.Config("many", 60 + B, B, [200 + 3 * i for i in range(B)], None, 0.02, n_q_heads=16, n_kv_heads=8, sparsity=4)
    w = wl.make_workload(cfg, DEV)
    Hq, Hkv = 16, 8
    shape = ha.make_shape(B, Hq, Hkv, w["sm_scale"])
    ws = ha.alloc_workspace(shape, w["n_cap"], w["k_max"])
    mq, mk = ha.Mapping(w["map_q"]), ha.Mapping(w["map_k"])
    kc = torch.zeros(B, Hkv, (w["n_cap"] + 3) // 4 * 4, dtype=torch.int32, device=DEV)
    ha.ha_encode(mk, 1, w["K"], kc)
    qc = torch.zeros(B, Hq, dtype=torch.int32, device=DEV)
    idx = torch.zeros(B, Hkv, w["k_max"], dtype=torch.int32, device=DEV)
    cnt = torch.zeros(B, Hkv, dtype=torch.int32, device=DEV)
    out = torch.zeros(B, Hq, 128, dtype=torch.bfloat16, device=DEV)
    ha.ha_sparse_decode(shape, mq, mk, w["q"], w["k_new"], w["K"], w["V"], kc, w["seq_lens"], w["k_per_seq"], 0,
                        w["n_cap"], w["k_max"], qc, idx, cnt, out, ws)
    kc_np = codes_np(kc)[:, :, :w["n_cap"]].copy()
    ref = oracle.decode_step(u16(w["q"]), u16(w["k_new"]), u16(w["K"]), u16(w["V"]), kc_np, wl.mapping_numpy(w["map_q"]),
                             wl.mapping_numpy(w["map_k"]), w["lens"], w["ks"], sm_scale=w["sm_scale"], n_threads=8)
    assert np.array_equal(idx.cpu().numpy(), ref["idx"]) and np.array_equal(cnt.cpu().numpy(), ref["count"])
    assert_out_close(u16(out), ref["out"])


@pytest.mark.parametrize("G", [2, 8])
def test_other_group_sizes_whole_step(G):
    cfg = wl.Config("g", 61 + G, 2, [5000, 777], None, 0.01, n_q_heads=2 * G, n_kv_heads=2, sparsity=8)
    w = wl.make_workload(cfg, DEV)
    B, Hq, Hkv = 2, 2 * G, 2
    shape = ha.make_shape(B, Hq, Hkv, w["sm_scale"])
    ws = ha.alloc_workspace(shape, w["n_cap"], w["k_max"])
    mq, mk = ha.Mapping(w["map_q"]), ha.Mapping(w["map_k"])
    kc = torch.zeros(B, Hkv, (w["n_cap"] + 3) // 4 * 4, dtype=torch.int32, device=DEV)
    ha.ha_encode(mk, 1, w["K"], kc)
    qc = torch.zeros(B, Hq, dtype=torch.int32, device=DEV)
    idx = torch.zeros(B, Hkv, w["k_max"], dtype=torch.int32, device=DEV)
    cnt = torch.zeros(B, Hkv, dtype=torch.int32, device=DEV)
    out = torch.zeros(B, Hq, 128, dtype=torch.bfloat16, device=DEV)
    ha.ha_sparse_decode(shape, mq, mk, w["q"], w["k_new"], w["K"], w["V"], kc, w["seq_lens"], w["k_per_seq"], 0,
                        w["n_cap"], w["k_max"], qc, idx, cnt, out, ws)
    kc_np = codes_np(kc)[:, :, :w["n_cap"]].copy()
    ref = oracle.decode_step(u16(w["q"]), u16(w["k_new"]), u16(w["K"]), u16(w["V"]), kc_np, wl.mapping_numpy(w["map_q"]),
                             wl.mapping_numpy(w["map_k"]), w["lens"], w["ks"], sm_scale=w["sm_scale"], n_threads=4)
    assert np.array_equal(codes_np(qc), ref["qcodes"])
    assert np.array_equal(idx.cpu().numpy(), ref["idx"]) and np.array_equal(cnt.cpu().numpy(), ref["count"])
    assert_out_close(u16(out), ref["out"])
