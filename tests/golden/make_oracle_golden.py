"""Writes tests/golden/oracle_tiny_forward.txt: the fp64 oracle's output on one tiny seeded input, kept so that an
accidental change of the oracle's arithmetic shows up as a diff.  Calls only the oracle and the seeded input generator.

    python tests/golden/make_oracle_golden.py
"""
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import cca_oracle as O                      # noqa: E402
from paper_2510_04476_b200 import synth                 # noqa: E402

SHAPE = synth.Shape("golden_tiny", 2, 7, 32, 4, 2, 4, k_seq=2, k_ch=2, seed=2510)


def compute():
    t = synth.make_inputs(SHAPE)
    cfg = O.OracleConfig(SHAPE.d_model, SHAPE.n_q_heads, SHAPE.n_kv_heads, SHAPE.head_dim, SHAPE.k_seq, SHAPE.k_ch,
                         SHAPE.causal, SHAPE.flags, SHAPE.rope_base)
    out, I = O.forward(cfg, t, t["x"])
    G = O.backward(cfg, t, I, t["d_out"])
    return {"out": out, "lse": I["lse"], "d_x": G["d_x"], "d_temp": G["d_temp"], "d_conv0_w": G["d_conv0_w"]}


def main():
    vals = compute()
    with open(os.path.join(HERE, "oracle_tiny_forward.txt"), "w") as f:
        f.write("# fp64 oracle on Shape(B=2, S=7, E=32, 4 q / 2 kv heads x 4, k_seq = k_ch = 2, seed 2510): written by\n")
        f.write("# tests/golden/make_oracle_golden.py (oracle only).  name, shape, then the values in row-major order.\n")
        for name, v in vals.items():
            f.write(f"{name} {' '.join(str(s) for s in v.shape)}\n")
            f.write(" ".join(repr(float(x)) for x in v.reshape(-1).tolist()) + "\n")


if __name__ == "__main__":
    main()
