"""The workspace-free score entry point (collected last on purpose).

lava_score_layer_static serves callers that cannot allocate device memory (code inside another
framework's pool, plugins barred from allocating after start-up, serving loops that must not
stall on an allocator): its scratch is a fixed array inside the library.  It must give what
lava_score_layer gives, call after call, although every call reuses the same scratch bytes.
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2509_09754_b200 as lava
from lava_workloads import get_config

SCORE_RTOL, SCORE_ATOL = 1e-3, 1e-6   # the tolerance of the score parity tests


def _one_layer(cfg):
    from tests.parity_harness import upload_model
    q, k, v, cu = upload_model(cfg)
    desc = lava.LayerDesc.for_tensors(q[0], k[0], v[0], cfg.window, cfg.pool_kind, cfg.pool_kernel,
                                      cu_seqlens=cu if cfg.batch > 1 else None,
                                      max_seqlen=max(cfg.seq_lens))
    return desc, q[0], k[0], v[0]


@pytest.mark.gpu
@pytest.mark.parametrize("name,kw", [
    ("llama8b_8k", dict(seq_lens=(1733,), n_layers=1)),          # tensor-core path
    ("tiny", dict()),                                            # CUDA-core path, fp32
    ("mistral7b_ragged", dict(seq_lens=(700, 1301), n_layers=1)),  # ragged batch
])
def test_static_scratch_matches_workspace_entry_point_twice(name, kw):
    cfg = get_config(name).scaled(**kw)
    desc, q, k, v = _one_layer(cfg)
    hkv = cfg.n_kv_heads
    ws = torch.zeros(lava.lava_workspace_bytes(desc, 1), dtype=torch.uint8, device="cuda")
    want_s = torch.empty(desc.total_scores, dtype=torch.float32, device="cuda")
    want_v = torch.empty((cfg.batch, hkv), dtype=torch.float32, device="cuda")
    want_e = torch.empty(cfg.batch, dtype=torch.float64, device="cuda")
    lava.lava_score_layer(desc, q, k, v, None, want_s, want_v, want_e, ws)
    for call in range(2):          # two calls in a row share the same built-in scratch
        got_s = torch.full_like(want_s, -1.0)
        got_v = torch.full_like(want_v, -1.0)
        got_e = torch.full_like(want_e, -1.0)
        status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
        lava.lava_score_layer_static(desc, q, k, v, None, got_s, got_v, got_e, status)
        torch.cuda.synchronize()
        assert int(status[0]) == 0
        np.testing.assert_allclose(got_s.cpu().numpy(), want_s.cpu().numpy(),
                                   rtol=SCORE_RTOL, atol=SCORE_ATOL)
        np.testing.assert_allclose(got_v.cpu().numpy(), want_v.cpu().numpy(), rtol=1e-5)
        np.testing.assert_allclose(got_e.cpu().numpy(), want_e.cpu().numpy(), rtol=1e-5)


def test_layers_beyond_the_built_in_scratch_are_rejected_on_the_host():
    """No GPU needed: the size check comes before any CUDA call."""
    n = 4 << 20   # 4M tokens: far more scratch than the 8 MiB array holds
    desc = lava.LayerDesc(n_q_heads=32, n_kv_heads=8, head_dim=128, window=32, total_tokens=n,
                          k_stride_head=n * 128, k_stride_tok=128, v_stride_head=n * 128,
                          v_stride_tok=128)
    assert lava.lava_workspace_bytes(desc, 1) > (8 << 20)
    c = desc.to_c()
    lib = lava.load_library()
    rc = lib.lava_score_layer_static(ctypes.byref(c), 16, 16, 16, None, 16, None, 16, None, None)
    assert rc == 3                                  # LAVA_ERR_WORKSPACE
    assert "built-in scratch" in lava.lava_last_error()
