"""Workload generator sanity and the oracle's stored output on the tiny workload."""
import os

import numpy as np
import torch

from lava_workloads import CONFIGS, generate_layer, get_config, to_numpy64
from lava_workloads.generate import needle_position, span_starts
from oracle import lava_oracle as O

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "tiny_config_oracle.txt")


def test_config_shapes_match_the_named_workloads():
    c = CONFIGS
    assert c["tiny"].total_budget() == 128
    assert c["llama8b_8k"].total_budget() == 512 * 8 * 32
    assert c["llama8b_32k"].total_budget() == 2048 * 8 * 32
    assert c["gqa7_128k"].group == 7 and c["gqa7_128k"].total_budget() == 1024 * 4 * 28
    lens = c["mistral7b_ragged"].seq_lens
    assert len(lens) == 8 and all(4096 <= n <= 16384 for n in lens) and len(set(lens)) > 1


def test_generation_is_seeded_and_structured():
    cfg = get_config("llama8b_8k").scaled(seq_lens=(700,), n_layers=2)
    a = generate_layer(cfg, 1, "cpu")
    b = generate_layer(cfg, 1, "cpu")
    c = generate_layer(cfg, 0, "cpu")
    assert torch.equal(a["k"], b["k"]) and torch.equal(a["v"], b["v"]) and torch.equal(a["q_win"], b["q_win"])
    assert not torch.equal(a["k"], c["k"])
    assert a["k"].dtype == torch.bfloat16 and a["k"].shape == (8, 700, 128)
    assert a["q_win"].shape == (1, 32, 32, 128)
    norms = a["v"].float().abs().sum(-1)
    assert norms.max() / norms.median() > 2.0            # log-normal row norms
    t = generate_layer(get_config("tiny"), 0, "cpu")
    kn = t["k"].norm(dim=-1)
    assert kn[:, :4].min() > 2.0 * kn[:, 4:].median()     # planted sinks


def test_ragged_needle_and_spans():
    cfg = get_config("mistral7b_ragged").scaled(seq_lens=(300, 257, 411), n_layers=1)
    t = generate_layer(cfg, 0, "cpu")
    assert t["cu_seqlens"].tolist() == [0, 300, 557, 968]
    assert t["k"].shape == (8, 968, 128) and t["q_win"].shape == (3, 32, 64, 128)
    for b in range(3):
        p = needle_position(cfg, b)
        assert 0 <= p < cfg.seq_lens[b] - cfg.window
    cfg5 = get_config("gqa7_128k").scaled(seq_lens=(4096,))
    st = span_starts(cfg5, 0)
    assert len(st) == 64 and all(st[i] + 16 <= st[i + 1] for i in range(63))


def test_oracle_reproduces_its_stored_tiny_output():
    cfg = get_config("tiny")
    t = generate_layer(cfg, 0, "cpu")
    q, k, v = to_numpy64(t["q_win"][0]), to_numpy64(t["k"]), to_numpy64(t["v"])
    s = O.lava_scores(q, k, v, cfg.window, cfg.pool_kind, cfg.pool_kernel)
    keep, off = O.select_topk(s, cfg.total_budget(), cfg.window)
    rows = {}
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#"):
                continue
            key, _, rest = line.strip().partition(" ")
            rows[key] = rest.split()
    assert abs(O.layer_entropy(s, 512) - float(rows["entropy"][0])) < 1e-12
    assert [int(x) for x in rows["head_offsets"]] == [int(x) for x in off]
    for g in range(2):
        assert [int(x) for x in rows["keep%d" % g]] == [int(x) for x in keep[g]]
        for item in rows["score%d" % g]:
            i, val = item.split(":")
            assert abs(s[g, int(i)] - float(val)) <= 1e-9 * abs(float(val))
    # the planted sinks (positions 0..3) survive in both heads
    for g in range(2):
        assert set(range(4)) <= set(int(x) for x in keep[g])
