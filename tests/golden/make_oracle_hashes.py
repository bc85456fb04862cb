"""Writes tests/golden/oracle_hashes.json: SHA-256 digests of seeded inputs and of what the CPU oracle
makes of them. Calls only the input generator and `oracle/` (never the CUDA library).

    python tests/golden/make_oracle_hashes.py

The digests pin the generator's bit streams and the oracle's arithmetic against later, unintended changes
(compiler flags, library versions); tests/test_oracle_pins.py recomputes and compares them.
"""
import hashlib
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2606_14598_b200 import inputs as synth  # noqa: E402

OUT = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_hashes.json")

# small cases with the structure of the benchmark configurations (outlier channels, GELU rows, ragged sizes)
CASES = [
    synth.LinearSpec("golden_c1", 128, 256, 256, outlier_frac=0.0),
    synth.LinearSpec("golden_outliers", 96, 3072, 264),
    synth.LinearSpec("golden_gelu", 40, 12288, 72, act="gelu", outlier_frac=0.0),
    synth.LinearSpec("golden_ragged", 33, 400, 136, bias=False),
]


def digest(a: np.ndarray) -> str:
    return hashlib.sha256(np.ascontiguousarray(a).tobytes()).hexdigest()


def compute(spec) -> dict:
    t = synth.make_linear(spec)
    A_bits = synth.bf16_bits(t["A"])
    W = t["W"].numpy()
    bias = None if t["bias"] is None else t["bias"].numpy()
    qw, s_ch = oracle.quantize_weight_per_channel(W)
    r = oracle.linear_fused_bf16(A_bits, qw, s_ch, bias)
    return {
        "shape": [spec.M, spec.K, spec.N],
        "A": digest(A_bits), "W": digest(W), "bias": None if bias is None else digest(bias),
        "qw": digest(qw), "s_ch": digest(s_ch), "qa": digest(r["qa"]), "s_tok": digest(r["s_tok"]),
        "acc": digest(r["acc"]), "out": digest(r["out"]),
    }


def compute_all() -> dict:
    return {spec.name: compute(spec) for spec in CASES}


if __name__ == "__main__":
    with open(OUT, "w") as f:
        json.dump(compute_all(), f, indent=1, sort_keys=True)
        f.write("\n")
    print("wrote", OUT)
