"""Oracle-side measurement behind the decision not to build prefix freezing.

TEST INFRASTRUCTURE ONLY (calls nothing but the CPU oracle).  By the induction step of Prop. 3.2, a position whose
inputs did not change in the last Jacobi sweep cannot change in this one, so its row could be dropped and its K/V
kept.  This script runs Algorithm 1 in fp64 on seeded models and prints, per sweep and sample, the first token index
whose value still changes by more than a threshold (0, 1e-7, 1.5e-5 = the resolution of a bf16 pair, 1e-4): the
length of the prefix that freezing could skip.

    python oracle/prefix_freeze_probe.py            (about two minutes of CPU)
"""
import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
from oracle import tarflow_oracle as O                      # noqa: E402
from paper_2505_24791_b200 import synth                     # noqa: E402


def probe(name, B, n_blocks, tau=1e-3, max_sweeps=12):
    cfg = synth.config(name, n_blocks=n_blocks)
    blocks = synth.make_weights(cfg)
    L = synth.seq_len(cfg)
    z = synth.make_latents(cfg, 1000, B=B)
    lab = synth.make_labels(cfg, B=B)
    seq = O.patchify(z.astype(np.float64), cfg["patch"])
    for g in range(n_blocks):
        v = np.ascontiguousarray(O.permute(seq, g))
        u = np.zeros_like(v)
        print(f"{name} block {g} ({L} tokens)")
        for t in range(1, max_sweeps):
            un = O.jacobi_map(blocks[g], u, v, lab, cfg)
            d = np.abs(un - u).max(axis=2)                  # [B, L]: largest change per token

            def first(thr):
                return [int(np.argmax(d[b] > thr)) if (d[b] > thr).any() else L for b in range(B)]

            print(f"  sweep {t}: max|du| = {d.max():.2e}   first changing token  >0: {first(0.0)}  >1e-7: {first(1e-7)}"
                  f"  >1.5e-5: {first(1.5e-5)}  >1e-4: {first(1e-4)}")
            u = un
            if d.max() <= tau:
                break
        seq = np.ascontiguousarray(O.permute(u, g))


if __name__ == "__main__":
    probe("cfg2", 3, 2)
    probe("cfg3", 2, 2)
