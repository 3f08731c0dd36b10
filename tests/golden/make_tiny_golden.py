"""Writes tests/golden/tiny_oracle.npz from the CPU oracle alone (run: python tests/golden/make_tiny_golden.py).

Stored: the oracle's outputs for the seeded Tiny workload and a SHA-256 of the input bytes they
were computed from, so that a machine whose random generator yields other bytes can tell.
"""
import hashlib
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from workloads import CONFIGS, bf16_bits, make_prompt  # noqa: E402


def input_digest(prompt) -> str:
    h = hashlib.sha256()
    h.update(bf16_bits(prompt.q).tobytes())
    for x in prompt.k:
        h.update(bf16_bits(x).tobytes())
    for t in (prompt.token_ids, prompt.char_start, prompt.char_end):
        h.update(t.numpy().tobytes())
    return h.hexdigest()


def main():
    prompt = make_prompt(CONFIGS["tiny"])
    cfg = prompt.cfg
    res = oracle.compress(bf16_bits(prompt.q), [bf16_bits(x) for x in prompt.k], prompt.token_ids.numpy(),
                          prompt.char_start.numpy(), prompt.char_end.numpy(), chunk=cfg.chunk,
                          keep=cfg.keep[0], pool_kernel=cfg.pool_kernel)
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tiny_oracle.npz")
    np.savez_compressed(out, digest=np.array(input_digest(prompt)), importance=res["importance"],
                        lse=res["lse"], chunk_scores=res["chunk_scores"], kept=res["kept"], ids=res["ids"],
                        pos=res["pos"], tok_spans=res["tok_spans"], char_spans=res["char_spans"])
    print("wrote", out)


if __name__ == "__main__":
    main()
