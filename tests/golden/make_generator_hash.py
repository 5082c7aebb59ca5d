"""Writes generator_sha256.txt: SHA-256 of the config-1 input arrays (weights 4096x4096, x[4096]).
Calls only numpy and the seeded input generator; freezes the generator against accidental change."""
import hashlib
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
from paper_2607_10183_b200 import workloads as W  # noqa: E402


def digests():
    packed, scales = W.q4_packed(1, 0, W.ROLE_Q, 4096, 4096)
    x = W.activations(1, 0, (1, 4096))
    return {"cfg1.packed": hashlib.sha256(packed.tobytes()).hexdigest(),
            "cfg1.scales": hashlib.sha256(scales.tobytes()).hexdigest(),
            "cfg1.x": hashlib.sha256(x.tobytes()).hexdigest()}


if __name__ == "__main__":
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "generator_sha256.txt"), "w") as f:
        for k, v in digests().items():
            f.write(f"{k} {v}\n")
