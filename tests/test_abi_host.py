"""Host-side checks of the C ABI: the library loads, exports every declared symbol, and
rejects bad arguments before any launch (no GPU needed)."""
import ctypes
import os
import re

import pytest

import paper_2509_09754_b200 as lava
from paper_2509_09754_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            names |= set(re.findall(r"LAVA_API[^;(]*?\b(lava_\w+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol():
    from paper_2509_09754_b200.build import build_library
    build_library()
    lib = lava.load_library()
    names = _declared_symbols()
    assert {"lava_score_layer", "lava_layer_budgets", "lava_select_topk", "lava_compact_kv"} <= names
    for name in names:
        assert hasattr(lib, name), name
    assert lava.lava_version() >= 100


def _desc(**kw):
    base = dict(n_q_heads=4, n_kv_heads=2, head_dim=64, window=16, total_tokens=512,
                k_stride_head=512 * 64, k_stride_tok=64, v_stride_head=512 * 64, v_stride_tok=64)
    base.update(kw)
    return lava.LayerDesc(**base)


@pytest.mark.parametrize("kw,status", [
    (dict(n_q_heads=5), 1), (dict(head_dim=96), 2), (dict(window=0), 1), (dict(window=200), 2),
    (dict(pool_kernel=4), 1), (dict(dtype=7), 1), (dict(batch=2), 1), (dict(total_tokens=8), 1),
    (dict(k_stride_tok=60), 1), (dict(k_stride_tok=32), 1), (dict(sm_scale=-1.0), 1),
])
def test_bad_geometry_is_rejected_on_the_host(kw, status):
    lib = lava.load_library()
    c = _desc(**kw).to_c()
    assert lib.lava_workspace_bytes(ctypes.byref(c), 1) == 0
    rc = lib.lava_score_layer(ctypes.byref(c), 16, 16, 16, None, 16, None, 16, 16, 1 << 30, None)
    assert rc == status
    assert len(lava.lava_last_error()) > 0


def test_null_misaligned_and_workspace_errors():
    lib = lava.load_library()
    c = _desc().to_c()
    need = lib.lava_workspace_bytes(ctypes.byref(c), 1)
    assert need > 256
    assert lib.lava_score_layer(ctypes.byref(c), None, 16, 16, None, 16, None, 16, 16, need, None) == 1
    assert lib.lava_score_layer(ctypes.byref(c), 16, 16, None, None, 16, None, 16, 16, need, None) == 1
    assert lib.lava_score_layer(ctypes.byref(c), 16, 24, 16, None, 16, None, 16, 16, need, None) == 1
    assert lib.lava_score_layer(ctypes.byref(c), 16, 16, 16, None, 16, None, 16, None, need, None) == 3
    assert lib.lava_score_layer(ctypes.byref(c), 16, 16, 16, None, 16, None, 16, 16, need - 1, None) == 3
    assert "workspace" in lava.lava_last_error()
    assert lib.lava_layer_budgets(0, 1, 16, 16, 16, 16, 0, 16, 16, None, None) == 2
    assert lib.lava_layer_budgets(4, 1, 16, 16, 16, 16, 9, 16, 16, None, None) == 1
    assert lib.lava_layer_budgets(4, 1, None, 16, 16, 16, 0, 16, 16, None, None) == 1
    assert lib.lava_select_topk(ctypes.byref(c), None, 16, 16, 16, None, 0, None) == 1
    assert lib.lava_compact_kv(ctypes.byref(c), 16, 16, 16, 16, 16, 24, 16, None) == 1
    assert lib.lava_compact_kv(None, 16, 16, 16, 16, 16, 16, 16, None) == 1
    assert lib.lava_wo_norm(16, 0, 0, 4, 16, None) == 1


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_LIB", None)
    monkeypatch.setattr(binding, "library_path", lambda: "/nonexistent/liblava.so")
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        binding.load_library()


def test_workspace_grows_with_layers_and_context():
    a = lava.lava_workspace_bytes(_desc(), 1)
    b = lava.lava_workspace_bytes(_desc(), 4)
    c = lava.lava_workspace_bytes(_desc(total_tokens=4096, k_stride_head=4096 * 64,
                                        v_stride_head=4096 * 64), 1)
    assert a < b and a < c


def _config_desc(name):
    from lava_workloads import get_config
    cfg = get_config(name)
    n, d = cfg.total_tokens, cfg.head_dim
    return cfg, lava.LayerDesc(
        n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads, head_dim=d, window=cfg.window,
        pool_kind=cfg.pool_kind, pool_kernel=cfg.pool_kernel,
        dtype=lava.LAVA_BF16 if cfg.dtype == "bf16" else lava.LAVA_F32, batch=cfg.batch,
        max_seqlen=max(cfg.seq_lens), cu_seqlens=None, total_tokens=n, k_stride_head=n * d,
        k_stride_tok=d, v_stride_head=n * d, v_stride_tok=d)


@pytest.mark.parametrize("name,path", [
    ("tiny", 0), ("llama8b_8k", 1), ("llama8b_32k", 1), ("gqa7_128k", 2)])
def test_which_kernels_score_each_workload(name, path):
    _, desc = _config_desc(name)
    assert lava.lava_score_path(desc) == path


def test_score_path_of_split_groups_and_of_what_stays_on_cuda_cores(monkeypatch):
    base = dict(head_dim=128, dtype=lava.LAVA_BF16, total_tokens=4096, k_stride_head=4096 * 128,
                k_stride_tok=128, v_stride_head=4096 * 128, v_stride_tok=128)
    mk = lambda **kw: lava.LayerDesc(**{**base, **kw})
    assert lava.lava_score_path(mk(n_q_heads=32, n_kv_heads=8, window=64)) == 2      # G 4 x w 64
    assert lava.lava_score_path(mk(n_q_heads=32, n_kv_heads=8, window=64,
                                   pool_kind=lava.LAVA_POOL_AVG, pool_kernel=5)) == 2
    assert lava.lava_score_path(mk(n_q_heads=32, n_kv_heads=2, window=16)) == 2      # 8 heads per unit
    assert lava.lava_score_path(mk(n_q_heads=32, n_kv_heads=8, window=128)) == 0     # 512 rows
    assert lava.lava_score_path(mk(n_q_heads=32, n_kv_heads=8, window=48)) == 0      # odd window
    assert lava.lava_score_path(mk(n_q_heads=32, n_kv_heads=2, window=16,
                                   pool_kind=lava.LAVA_POOL_AVG, pool_kernel=5)) == 0  # avg: > 4 heads
    assert lava.lava_score_path(mk(n_q_heads=32, n_kv_heads=8, window=32, dtype=lava.LAVA_F32)) == 0
    lava.lava_set_option("force_generic", 1)
    try:
        assert lava.lava_score_path(mk(n_q_heads=32, n_kv_heads=8, window=32)) == 0
    finally:
        lava.lava_set_option("force_generic", 0)
    assert lava.lava_score_path(mk(n_q_heads=32, n_kv_heads=8, window=32)) == 1
    with pytest.raises(lava.LavaError):
        lava.lava_score_path(mk(n_q_heads=5, n_kv_heads=2, window=32))


def test_workspace_for_a_model_also_serves_single_layers():
    _, desc = _config_desc("llama8b_32k")
    assert lava.lava_workspace_bytes(desc, 32) >= lava.lava_workspace_bytes(desc, 1)
    assert lava.lava_workspace_bytes(desc, 32) >= lava.lava_workspace_bytes(desc, 7)


def test_options_round_trip_and_reject_bad_values():
    for name, value in (("select_cluster", 16), ("score_chunk_tiles", 8), ("score_lead_tiles", 5),
                        ("wait_limit_cycles", 12345), ("score_kernel", 1)):
        before = lava.lava_get_option(name)
        lava.lava_set_option(name, value)
        assert lava.lava_get_option(name) == value
        lava.lava_set_option(name, before)
        assert lava.lava_get_option(name) == before
    lib = lava.load_library()
    assert lib.lava_set_option(b"select_cluster", 12) == 1
    assert lib.lava_set_option(b"wait_limit_cycles", 0) == 1
    assert lib.lava_set_option(b"no_such_option", 1) == 1
    assert lib.lava_set_option(None, 1) == 1
    assert "unknown option" in lava.lava_last_error()
    with pytest.raises(lava.LavaError):
        lava.lava_get_option("no_such_option")


def test_host_buffer_arena_size_ignores_the_descriptor_strides():
    """The host arrays of lava_evict_model_host are dense, so whatever strides the descriptor
    carries (zeros included) must give the same arena size."""
    cfg, desc = _config_desc("llama8b_8k")
    dense = lava.lava_host_arena_bytes(desc, 4, 4 * 8 * 512)
    import dataclasses
    zero = dataclasses.replace(desc, k_stride_head=0, k_stride_tok=0, v_stride_head=0, v_stride_tok=0)
    odd = dataclasses.replace(desc, k_stride_tok=1024, v_stride_tok=256, k_stride_head=8)
    assert dense > 0
    assert lava.lava_host_arena_bytes(zero, 4, 4 * 8 * 512) == dense
    assert lava.lava_host_arena_bytes(odd, 4, 4 * 8 * 512) == dense
