"""ha_gather_attn_static — the entry point for callers that cannot allocate a workspace (for
instance a process whose memory pool already owns the whole GPU, or a plug-in that may only launch
kernels): its scratch is a fixed array inside the library.  The test calls it through the C ABI
twice in a row, on different inputs, and compares each result with ha_gather_attn (which uses a
caller-allocated workspace) and, head by head, with the CPU oracle's GATHER-ATT, within the
tolerance of the other attention tests; the second call shows that what the first one left in the
shared array does no harm.  This file sorts last so that a
run that stops at the first failure has already run everything else; it also passes on its own."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2412_14468_b200 import binding as ha
from tests._util import assert_out_close, u16

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _case(seed, B, Hq, Hkv, n_cap, k_max):
    g = torch.Generator(DEV).manual_seed(seed)
    q = torch.randn(B, Hq, 128, device=DEV, generator=g).to(torch.bfloat16)
    K = torch.randn(B, Hkv, n_cap, 128, device=DEV, generator=g).to(torch.bfloat16)
    V = torch.randn(B, Hkv, n_cap, 128, device=DEV, generator=g).to(torch.bfloat16)
    lens = [n_cap - 7 * b for b in range(B)]
    rng = np.random.default_rng(seed)
    idx = np.full((B, Hkv, k_max), -1, np.int32)
    cnt = np.zeros((B, Hkv), np.int32)
    for b in range(B):
        for h in range(Hkv):
            c = int(rng.integers(0, k_max + 1)) if (b + h) % 3 else k_max      # mixes full, partial and empty lists
            cnt[b, h] = c
            idx[b, h, :c] = np.sort(rng.choice(lens[b], size=c, replace=False))
    return q, K, V, torch.tensor(lens, dtype=torch.int32, device=DEV), torch.from_numpy(idx).to(DEV), \
        torch.from_numpy(cnt).to(DEV)


def test_static_scratch_entry_matches_workspace_entry_on_two_calls_in_a_row():
    B, Hq, Hkv = 2, 32, 8
    shape = ha.make_shape(B, Hq, Hkv, 1.0 / math.sqrt(128))
    ws = ha.alloc_workspace(shape, 40000, 2048)
    for seed, n_cap, k_max in ((901, 40000, 2048), (902, 9000, 700)):       # many parts per unit, then few
        q, K, V, sl, idx, cnt = _case(seed, B, Hq, Hkv, n_cap, k_max)
        ref = torch.full((B, Hq, 128), 5.0, dtype=torch.bfloat16, device=DEV)
        got = torch.full((B, Hq, 128), -5.0, dtype=torch.bfloat16, device=DEV)
        lse_ref = torch.zeros(B, Hq, device=DEV)
        lse_got = torch.ones(B, Hq, device=DEV)
        ha.ha_gather_attn(shape, q, K, V, sl, idx, cnt, k_max, ref, ws, lse=lse_ref)
        ha.ha_gather_attn_static(shape, q, K, V, sl, idx, cnt, k_max, got, lse=lse_got)
        torch.cuda.synchronize()
        assert_out_close(u16(got), u16(ref))
        both_inf = torch.isinf(lse_ref) & torch.isinf(lse_got)
        assert torch.equal(torch.isinf(lse_ref), torch.isinf(lse_got))
        assert float(((lse_ref - lse_got).abs()[~both_inf]).max()) < 1e-4
        # ... and directly against the oracle, one query head at a time
        qu, Ku, Vu, got_u, idx_np, cnt_np = u16(q), u16(K), u16(V), u16(got), idx.cpu().numpy(), cnt.cpu().numpy()
        lse_np = lse_got.cpu().numpy()
        G = Hq // Hkv
        for b in range(B):
            for h in range(Hq):
                g = h // G
                eo, el, _ = oracle.gather_attn(qu[b, h], Ku[b, g], Vu[b, g], idx_np[b, g, :cnt_np[b, g]],
                                               sm_scale=1.0 / math.sqrt(128), n_valid=int(sl[b]))
                assert_out_close(got_u[b, h], eo)
                assert (np.isneginf(el) and np.isneginf(lse_np[b, h])) or abs(float(lse_np[b, h]) - el) < 1e-3


def test_static_scratch_entry_rejects_problems_beyond_its_limit():
    B, Hq, Hkv = 9, 32, 8                                                      # 72 units > 64
    shape = ha.make_shape(B, Hq, Hkv, 0.1)
    q, K, V, sl, idx, cnt = _case(903, B, Hq, Hkv, 64, 8)
    out = torch.zeros(B, Hq, 128, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(ha.HashAttnError) as e:
        ha.ha_gather_attn_static(shape, q, K, V, sl, idx, cnt, 8, out)
    assert e.value.status == ha.HA_ERR_STATIC_LIMIT and "built-in scratch" in str(e.value)
