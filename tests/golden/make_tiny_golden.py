"""Writes tests/golden/tiny_config_oracle.txt from the oracle alone (no CUDA code involved).

Run:  python tests/golden/make_tiny_golden.py
The file stores, for the tiny fp32 workload (4 query / 2 KV heads, d 64, n 512, w 16, max-pool
5, layer budget 128), the oracle's layer entropy, per-head retained counts, the kept prefix
positions and 16 sampled scores.  It guards the oracle against accidental edits; the values are
the oracle's own, not the paper's (the paper prints no worked example).
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from lava_workloads import generate_layer, get_config, to_numpy64  # noqa: E402
from oracle import lava_oracle as O  # noqa: E402


def main():
    cfg = get_config("tiny")
    t = generate_layer(cfg, 0, "cpu")
    q, k, v = to_numpy64(t["q_win"][0]), to_numpy64(t["k"]), to_numpy64(t["v"])
    s = O.lava_scores(q, k, v, cfg.window, cfg.pool_kind, cfg.pool_kernel)
    e = O.layer_entropy(s, cfg.seq_lens[0])
    keep, off = O.select_topk(s, cfg.total_budget(), cfg.window)
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_config_oracle.txt")
    with open(path, "w") as f:
        f.write("# oracle output on the tiny workload; written by make_tiny_golden.py\n")
        f.write("entropy %.17e\n" % e)
        f.write("head_offsets %s\n" % " ".join(str(int(x)) for x in off))
        for g in range(cfg.n_kv_heads):
            f.write("keep%d %s\n" % (g, " ".join(str(int(x)) for x in keep[g])))
        idx = np.linspace(0, s.shape[1] - 1, 16).astype(int)
        for g in range(cfg.n_kv_heads):
            f.write("score%d %s\n" % (g, " ".join("%d:%.17e" % (i, s[g, i]) for i in idx)))
    print("wrote", path)


if __name__ == "__main__":
    main()
