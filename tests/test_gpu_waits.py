"""Device-side failure reporting without faulting or hanging anything.

Every wait inside the score kernels is bounded.  With the limit set to a few hundred cycles some
wait on another role or CTA runs out: the kernel must still return, the status word must carry
LAVA_DEV_WAIT_EXPIRED, lava_poll_status must turn that into LAVA_ERR_TIMEOUT, and the next call
with the normal limit, on the same workspace, must be correct again.  (Waits for copies that are
already in flight keep their long limit, so no CTA leaves under a running copy.)

A batch with a sequence shorter than the window has no room in the score layout: both score
paths flag it with LAVA_DEV_SHORT_SEQUENCE and write nothing.
"""
import numpy as np
import pytest
import torch

import paper_2509_09754_b200 as lava
from lava_workloads import get_config, to_numpy64
from oracle import lava_oracle as O
from tests.parity_harness import SCORE_ATOL, SCORE_RTOL, upload_model

pytestmark = pytest.mark.gpu

LAVA_DEV_SHORT_SEQUENCE, LAVA_DEV_WAIT_EXPIRED = 1, 4


def _score_once(desc, q, k, v, ws):
    hkv = desc.n_kv_heads
    sc = torch.zeros(desc.total_scores, dtype=torch.float32, device="cuda")
    vb = torch.zeros((desc.batch, hkv), dtype=torch.float32, device="cuda")
    ent = torch.zeros(desc.batch, dtype=torch.float64, device="cuda")
    lava.lava_score_layer(desc, q, k, v, None, sc, vb, ent, ws)
    return sc, vb, ent


@pytest.mark.parametrize("kernel", [1, 2])
def test_expired_wait_is_reported_and_the_next_call_is_correct(kernel):
    cfg = get_config("llama8b_8k").scaled(seq_lens=(2000,), n_layers=1)
    q, k, v, cu = upload_model(cfg)
    desc = lava.LayerDesc.for_tensors(q[0], k[0], v[0], cfg.window, cfg.pool_kind, cfg.pool_kernel,
                                      max_seqlen=2000)
    ws = torch.zeros(lava.lava_workspace_bytes(desc, 1), dtype=torch.uint8, device="cuda")
    normal = lava.lava_get_option("wait_limit_cycles")
    lava.lava_set_option("score_kernel", kernel)
    try:
        lava.lava_set_option("wait_limit_cycles", 300)
        _score_once(desc, q[0], k[0], v[0], ws)
        with pytest.raises(lava.LavaError) as err:
            lava.lava_poll_status(ws)
        assert err.value.status == 5                       # LAVA_ERR_TIMEOUT
        lava.lava_set_option("wait_limit_cycles", normal)
        assert lava.lava_poll_status(ws) == 0              # the poll above cleared the word
        sc, vb, ent = _score_once(desc, q[0], k[0], v[0], ws)
        assert lava.lava_poll_status(ws) == 0
        want = O.lava_scores(to_numpy64(q[0, 0]), to_numpy64(k[0]), to_numpy64(v[0]), cfg.window,
                             cfg.pool_kind, cfg.pool_kernel)
        got = sc.cpu().numpy().reshape(want.shape).astype(np.float64)
        assert np.all(np.abs(got - want) <= SCORE_RTOL * np.abs(want) + SCORE_ATOL)
    finally:
        lava.lava_set_option("wait_limit_cycles", normal)
        lava.lava_set_option("score_kernel", 0)


@pytest.mark.parametrize("generic", [0, 1])
def test_short_sequence_sets_the_status_bit(generic):
    cfg = get_config("llama8b_8k").scaled(seq_lens=(700, 20, 900), n_layers=1)
    q, k, v, cu = upload_model(cfg)
    desc = lava.LayerDesc.for_tensors(q[0], k[0], v[0], cfg.window, cfg.pool_kind, cfg.pool_kernel,
                                      cu_seqlens=cu, max_seqlen=900)
    ws = torch.zeros(lava.lava_workspace_bytes(desc, 1), dtype=torch.uint8, device="cuda")
    lava.lava_set_option("force_generic", generic)
    try:
        assert lava.lava_score_path(desc) == (0 if generic else 1)
        w, hkv = cfg.window, cfg.n_kv_heads
        sc = torch.full((hkv * (cfg.total_tokens - 3 * w),), -7.0, dtype=torch.float32, device="cuda")
        vb = torch.zeros((3, hkv), dtype=torch.float32, device="cuda")
        ent = torch.zeros(3, dtype=torch.float64, device="cuda")
        lava.lava_score_layer(desc, q[0], k[0], v[0], None, sc, vb, ent, ws)
        status = lava.lava_poll_status(ws)
        assert status & LAVA_DEV_SHORT_SEQUENCE
        assert not status & LAVA_DEV_WAIT_EXPIRED
        # The short sequence's n - w is negative, so its neighbours' score arrays would overlap and
        # the last one would run past the end of the layer: nothing may be written.
        assert bool((sc == -7.0).all())
    finally:
        lava.lava_set_option("force_generic", 0)
