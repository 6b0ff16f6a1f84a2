"""Writes tests/golden/bench_inputs_sha256.txt: the SHA-256 of every synthetic input tensor
of the benchmark step (both LLaMA-7B MLP shapes; the batch is rank 0's), drawn by
paper_2309_14717_b200.synthetic alone.  bench.py hashes the tensors it actually uses and
reports whether they match this record, so that a library version drawing different numbers
from the same seeds is noticed.

    python tests/golden/make_bench_inputs_sha256.py
"""
import hashlib
import os
import sys

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from paper_2309_14717_b200.synthetic import CONFIGS, make_inputs  # noqa: E402


def digest(t):
    t = t.contiguous()
    if t.dtype == torch.bfloat16:
        t = t.view(torch.int16)
    return hashlib.sha256(t.numpy().tobytes()).hexdigest()


def main():
    lines = ["# shape tensor sha256   (torch " + torch.__version__ + "; batch of rank 0: seed + 1000)"]
    for name in ("cfg3_7b_up", "cfg3_7b_down"):
        cfg = CONFIGS[name]
        shared = make_inputs(cfg, need=("W", "A", "B"))
        batch = make_inputs(cfg.with_(seed=cfg.seed + 1000), need=("x", "dy"))
        for k in ("W", "A", "B"):
            lines.append(f"{name} {k} {digest(shared[k])}")
        for k in ("x", "dy"):
            lines.append(f"{name} {k} {digest(batch[k])}")
    with open(os.path.join(HERE, "bench_inputs_sha256.txt"), "w") as f:
        f.write("\n".join(lines) + "\n")
    print("\n".join(lines))


if __name__ == "__main__":
    main()
