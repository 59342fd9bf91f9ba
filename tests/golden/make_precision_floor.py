"""Writes tests/golden/precision_floor.txt: how far the oracle's logits move when only its accumulation
precision changes (float32 vs float64), per configuration.  Calls nothing but the oracle and the input
generator.  Any two implementations of the same bf16-rounding contract whose summation order differs
decorrelate at the rounding points (a value within summation error of a rounding boundary flips, the
flip perturbs everything downstream, which flips more), so this figure is the floor for logits parity of
a deep configuration.  Usage: python tests/golden/make_precision_floor.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
import seeded_inputs as si  # noqa: E402
from oracle.forward import OracleModel  # noqa: E402


def main():
    lines = ["# config  steps  logit_std  max_abs_diff  mean_abs_diff  mean_rel_diff   (oracle float32 vs float64, prefill + steps-1 decode, teacher-forced)"]
    for c, n_dec in ((1, 16), (2, 3)):
        cfg = si.CONFIGS[c]
        lay = si.build_layout(cfg)
        W = si.weights_as_bits(lay)
        prompt = si.prompt_tokens(cfg)
        ref, toks = OracleModel(cfg, W, dtype=np.float64).generate(prompt, n_dec)
        got, _ = OracleModel(cfg, W, dtype=np.float32).generate(prompt, n_dec, forced=toks)
        mx = max(float(np.abs(a - b).max()) for a, b in zip(got, ref))
        mean = float(np.mean([np.abs(a - b).mean() for a, b in zip(got, ref)]))
        rel = max(float(np.abs(a - b).mean() / np.abs(b).mean()) for a, b in zip(got, ref))
        lines.append(f"{c} {n_dec + 1} {float(ref[0].std()):.6f} {mx:.6f} {mean:.6f} {rel:.6f}")
        print(lines[-1], flush=True)
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "precision_floor.txt"), "w") as f:
        f.write("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()
