"""Boundary tests that need no GPU: the C-ABI library loads, exports every function the header
declares, sizes its workspace on the host, and rejects bad arguments with error codes before
touching CUDA."""
import ctypes as C
import os
import re

import pytest

from paper_2412_14468_b200 import binding as ha
from paper_2412_14468_b200 import build as ha_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    ha_build.build()
    return ha.lib()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "hashattn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ha_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert set(names) == set(ha.EXPORTS), (names, ha.EXPORTS)
    for n in names:
        assert hasattr(lib, n), n


def test_binding_has_same_names():
    for n in ha.EXPORTS:
        if n == "ha_status_string":
            assert hasattr(ha, "status_string")
        else:
            assert hasattr(ha, n), n


def test_version_and_status_strings(lib):
    assert "sm_100a" in ha.ha_version()
    assert ha.status_string(0) == "ok"
    assert len({ha.status_string(i) for i in range(6)}) == 6


def test_workspace_bytes_is_host_only_and_monotone_in_batch(lib):
    s1 = ha.make_shape(1, 32, 8, 0.088)
    s16 = ha.make_shape(16, 32, 8, 0.088)
    a, b = ha.ha_workspace_bytes(s1, 32768, 1024), ha.ha_workspace_bytes(s16, 32768, 2048)
    assert 0 < a < b and a % 256 == 0
    long_seq = ha.ha_workspace_bytes(s1, 524288, 16384)             # + one score byte per token and KV head
    assert a + 8 * (524288 - 32768) <= long_seq <= a + 8 * 524288
    for bad in (ha.make_shape(1, 32, 8, 0.1, head_dim=64), ha.make_shape(1, 30, 8, 0.1), ha.make_shape(1, 24, 8, 0.1),
                ha.make_shape(-1, 32, 8, 0.1)):
        assert lib.ha_workspace_bytes(C.byref(bad), 100, 10) == 0


def test_bad_arguments_are_rejected_on_the_host(lib):
    s = ha.make_shape(1, 32, 8, 0.088)
    fake = 0x1000          # never dereferenced: validation fails first
    # NULL pointers
    assert lib.ha_score_topk(C.byref(s), None, fake, 0, 0, fake, None, 4, 16, 4, fake, 0, 0, fake, None, fake, 1 << 30, None) \
        == ha.HA_ERR_INVALID_ARG
    # unsupported head_dim
    s64 = ha.make_shape(1, 32, 8, 0.1, head_dim=64)
    assert lib.ha_score_topk(C.byref(s64), fake, fake, 0, 0, fake, None, 4, 16, 4, fake, 0, 0, fake, None, fake, 1 << 30, None) \
        == ha.HA_ERR_UNSUPPORTED
    # misaligned code cache row stride
    assert lib.ha_score_topk(C.byref(s), fake, fake, 6, 3, fake, None, 4, 16, 4, fake, 0, 0, fake, None, fake, 1 << 30, None) \
        == ha.HA_ERR_INVALID_ARG
    # workspace too small / misaligned / missing
    assert lib.ha_score_topk(C.byref(s), fake, fake, 16, 16, fake, None, 4, 16, 4, fake, 0, 0, fake, None, fake, 512, None) \
        == ha.HA_ERR_WORKSPACE
    assert lib.ha_score_topk(C.byref(s), fake, fake, 16, 16, fake, None, 4, 16, 4, fake, 0, 0, fake, None, fake + 8, 1 << 30, None) \
        == ha.HA_ERR_WORKSPACE
    assert lib.ha_score_topk(C.byref(s), fake, fake, 16, 16, fake, None, 4, 16, 4, fake, 0, 0, fake, None, None, 0, None) \
        == ha.HA_ERR_WORKSPACE
    # negative budget
    assert lib.ha_score_topk(C.byref(s), fake, fake, 16, 16, fake, None, -1, 16, 4, fake, 0, 0, fake, None, fake, 1 << 30, None) \
        == ha.HA_ERR_INVALID_ARG
    # mapping with the wrong widths / tensors with bad strides
    m = ha.ha_mapping(8, 128, 64, 32, fake, fake, fake, None, None, None)
    t = ha.ha_tensor(fake, 1024, 128, 128)
    assert lib.ha_encode(C.byref(m), 1, C.byref(t), 1, 8, 1, fake, 8, 1, None, None) == ha.HA_ERR_UNSUPPORTED
    m = ha.ha_mapping(8, 128, 128, 32, fake, fake, fake, None, None, None)
    tbad = ha.ha_tensor(fake, 1024, 128, 100)
    assert lib.ha_encode(C.byref(m), 1, C.byref(tbad), 1, 8, 1, fake, 8, 1, None, None) == ha.HA_ERR_INVALID_ARG
    assert lib.ha_encode(C.byref(m), 3, C.byref(t), 1, 8, 1, fake, 8, 1, None, None) == ha.HA_ERR_INVALID_ARG
    assert lib.ha_gather_attn(C.byref(s), fake, C.byref(tbad), C.byref(t), fake, fake, 0, 0, fake, 4, fake, None, fake, 1 << 30, None) \
        == ha.HA_ERR_INVALID_ARG
    assert lib.ha_dense_decode(C.byref(s), None, C.byref(t), C.byref(t), fake, 16, fake, None, fake, 1 << 30, None) \
        == ha.HA_ERR_INVALID_ARG
    # empty batch is a no-op that succeeds without touching the device
    s0 = ha.make_shape(0, 32, 8, 0.088)
    assert lib.ha_dense_decode(C.byref(s0), fake, C.byref(t), C.byref(t), fake, 16, fake, None, fake, 1 << 30, None) == ha.HA_OK


def test_windows_and_prefill_arguments_are_checked_on_the_host(lib):
    fake = 0x1000
    # always-kept windows: negative sizes, and windows that do not fit the index rows
    neg = ha.make_shape(1, 32, 8, 0.088, n_sink=-1)
    assert lib.ha_score_topk(C.byref(neg), fake, fake, 16, 16, fake, None, 4, 16, 4, fake, 0, 0, fake, None, fake, 1 << 30, None) \
        == ha.HA_ERR_INVALID_ARG
    wide = ha.make_shape(1, 32, 8, 0.088, n_sink=128, n_local=128)
    assert lib.ha_score_topk(C.byref(wide), fake, fake, 16, 16, fake, None, 4, 4096, 255, fake, 0, 0, fake, None, fake, 1 << 30, None) \
        == ha.HA_ERR_INVALID_ARG
    assert ha.ha_workspace_bytes(wide, 32768, 1280) == ha.ha_workspace_bytes(ha.make_shape(1, 32, 8, 0.088), 32768, 1280)
    # prompt encoder: unknown path, misaligned workspace, mismatching head counts; an empty call succeeds
    m = ha.ha_mapping(8, 128, 128, 32, fake, fake, fake, None, None, None)
    t = ha.ha_tensor(fake, 1 << 20, 1 << 16, 128)
    assert lib.ha_encode_prefill(C.byref(m), 1, C.byref(t), 1, 8, 64, fake, 64, 64, 7, None, None) == ha.HA_ERR_INVALID_ARG
    assert lib.ha_encode_prefill(C.byref(m), 1, C.byref(t), 1, 8, 64, fake, 64, 64, ha.HA_PREFILL_TCGEN05, fake + 8, None) \
        == ha.HA_ERR_WORKSPACE
    assert lib.ha_encode_prefill(C.byref(m), 4, C.byref(t), 1, 8, 64, fake, 64, 64, ha.HA_PREFILL_MMA_SYNC, None, None) \
        == ha.HA_ERR_INVALID_ARG
    assert lib.ha_encode_prefill(C.byref(m), 1, C.byref(t), 1, 8, 0, fake, 64, 64, ha.HA_PREFILL_TCGEN05, None, None) == ha.HA_OK


def test_summed_group_score_arguments_are_checked_on_the_host(lib):
    fake = 0x1000
    s = ha.make_shape(1, 32, 8, 0.088)
    call = lambda shape, q=fake, k=fake, sb=16, sh=16, lens=fake, k_uni=4, k_max=4, idx=fake, cnt=fake: \
        lib.ha_score_topk_sum(C.byref(shape), q, k, sb, sh, lens, None, k_uni, k_max, idx, 0, 0, cnt, None, None)
    assert call(s, q=None) == ha.HA_ERR_INVALID_ARG
    assert call(s, idx=None) == ha.HA_ERR_INVALID_ARG
    assert call(s, k=fake + 4) == ha.HA_ERR_INVALID_ARG          # signature rows not 16-byte aligned
    assert call(s, sh=18) == ha.HA_ERR_INVALID_ARG
    assert call(s, k_uni=-1) == ha.HA_ERR_INVALID_ARG
    assert call(s, k_max=-1) == ha.HA_ERR_INVALID_ARG
    assert call(ha.make_shape(1, 32, 8, 0.088, n_sink=128, n_local=128), k_max=255) == ha.HA_ERR_INVALID_ARG
    assert call(ha.make_shape(1, 32, 5, 0.088)) in (ha.HA_ERR_INVALID_ARG, ha.HA_ERR_UNSUPPORTED)   # heads do not divide
    assert call(ha.make_shape(0, 32, 8, 0.088)) == ha.HA_OK      # empty batch: no launch


def test_per_query_head_arguments_are_checked_on_the_host(lib):
    fake = 0x1000
    s = ha.make_shape(2, 32, 8, 0.088)
    t = ha.ha_tensor(fake, 1 << 20, 1 << 16, 128)
    sel = lambda shape, q=fake, k=fake, k_max=4, idx=fake: \
        lib.ha_score_topk_per_head(C.byref(shape), q, k, 16, 16, fake, None, 4, k_max, idx, 0, 0, fake, None, None)
    assert sel(s, q=None) == ha.HA_ERR_INVALID_ARG
    assert sel(s, idx=None) == ha.HA_ERR_INVALID_ARG
    assert sel(s, k=fake + 4) == ha.HA_ERR_INVALID_ARG
    assert sel(s, k_max=-1) == ha.HA_ERR_INVALID_ARG
    assert sel(ha.make_shape(4096, 32, 8, 0.088)) == ha.HA_ERR_UNSUPPORTED      # more than 65536 query-head units
    assert sel(ha.make_shape(0, 32, 8, 0.088)) == ha.HA_OK
    att = lambda shape, q=fake, ws=fake, nbytes=1 << 30: \
        lib.ha_gather_attn_per_head(C.byref(shape), q, C.byref(t), C.byref(t), fake, fake, 0, 0, fake, 4, fake, None, ws, nbytes, None)
    assert att(s, q=None) == ha.HA_ERR_INVALID_ARG
    assert att(s, ws=None) == ha.HA_ERR_WORKSPACE
    # the scratch is laid out for one unit per query head: its size is that of the shape with n_kv_heads = n_q_heads
    per_head = ha.ha_workspace_bytes(ha.make_shape(2, 32, 32, 0.088), 0, 64)
    assert att(s, nbytes=per_head - 256) == ha.HA_ERR_WORKSPACE
    assert att(ha.make_shape(0, 32, 8, 0.088), nbytes=per_head) == ha.HA_OK


def test_wide_score_and_inner_product_arguments_are_checked_on_the_host(lib):
    fake = 0x1000
    assert lib.ha_score_wide(fake, fake, 100, 96, fake, None) == ha.HA_ERR_UNSUPPORTED        # width not 64/128/256/512
    assert lib.ha_score_wide(fake, fake, -1, 64, fake, None) == ha.HA_ERR_INVALID_ARG
    assert lib.ha_score_wide(fake, fake + 8, 100, 128, fake, None) == ha.HA_ERR_INVALID_ARG   # signatures not 16-byte aligned
    assert lib.ha_score_wide(fake, fake, 100, 64, fake + 2, None) == ha.HA_ERR_INVALID_ARG    # scores not 4-byte aligned
    assert lib.ha_score_wide(None, fake, 100, 64, fake, None) == ha.HA_ERR_INVALID_ARG
    assert lib.ha_score_wide(fake, None, 0, 512, None, None) == ha.HA_OK                      # empty: no launch
    assert lib.ha_inner_products(fake, fake, 10, 100, fake, None) == ha.HA_ERR_INVALID_ARG    # rows shorter than 128
    assert lib.ha_inner_products(fake, fake, 10, 132, fake, None) == ha.HA_ERR_INVALID_ARG    # row stride not a multiple of 8
    assert lib.ha_inner_products(fake, fake + 4, 10, 128, fake, None) == ha.HA_ERR_INVALID_ARG
    assert lib.ha_inner_products(fake, None, 0, 128, None, None) == ha.HA_OK


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(ha, "_lib", None)
    monkeypatch.setattr(ha, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        ha.lib()
