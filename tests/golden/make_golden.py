"""Writes tests/golden/*.txt from the seeded generators and the CPU oracle only (never from the CUDA path).

    python tests/golden/make_golden.py

The paper prints no numeric worked example of a GEMM or attention result, so these files pin (a) the seeded
input generators (first BF16 bit patterns and a checksum of each benchmark tensor family on a small shape) and
(b) the oracle's output on one tiny fixed case, against silent drift of either.
"""
import hashlib
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle  # noqa: E402
from paper_2503_14985_b200 import inputs  # noqa: E402


def inputs_lines():
    out = []
    A, B = inputs.gemm_inputs(8, 8, 8, seed=0, kind="uniform")
    out.append("gemm uniform seed0 A[0,:8] " + " ".join(f"{v:04x}" for v in A[0]))
    out.append("gemm uniform seed0 B[0,:8] " + " ".join(f"{v:04x}" for v in B[0]))
    A, B = inputs.gemm_inputs(64, 48, 32, seed=1, kind="normal")
    out.append("gemm normal seed1 64x48x32 sha256 " + hashlib.sha256(A.tobytes() + B.tobytes()).hexdigest())
    Q, K, V = inputs.mha_inputs(1, 2, 16, 24, 64, seed=6, outlier_percent=1)
    out.append("mha seed6 1x2x16x24x64 outliers sha256 " + hashlib.sha256(Q.tobytes() + K.tobytes() + V.tobytes()).hexdigest())
    out.append("mha seed6 Q[0,0,0,:8] " + " ".join(f"{v:04x}" for v in Q[0, 0, 0, :8]))
    A, B, C = inputs.gemm_f16_inputs(8, 8, 8, seed=3, kind="normal")
    out.append("gemm_f16 normal seed3 A[0,:8] " + " ".join(f"{v:04x}" for v in A[0]))
    out.append("gemm_f16 normal seed3 sha256 " + hashlib.sha256(A.tobytes() + B.tobytes() + C.tobytes()).hexdigest())
    Qp, Kc, Vc, table, lens = inputs.paged_inputs(3, 4, 2, 64, 8, seed=9, min_len=5, max_len=40)[:5]
    out.append("paged seed9 sha256 " + hashlib.sha256(Qp.tobytes() + Kc.tobytes() + Vc.tobytes() + table.tobytes() + lens.tobytes()).hexdigest())
    return out


def oracle_lines():
    out = []
    A, B = inputs.gemm_inputs(3, 4, 5, seed=0, kind="uniform", lda=8, ldb=8)
    C = oracle.gemm(A, B, 3, 4, 5)
    for row in C:
        out.append("gemm 3x4x5 " + " ".join(float(v).hex() for v in row))
    Q, K, V = inputs.mha_inputs(1, 1, 3, 5, 4, seed=4)
    O, L = oracle.mha_fwd(Q, K, V, causal=True, scale=np.float32(0.5))
    for row, l in zip(O, L):
        out.append("mha 3x5x4 causal " + " ".join(float(v).hex() for v in row) + " lse " + float(l).hex())
    A, B, C0 = inputs.gemm_f16_inputs(3, 4, 5, seed=2, kind="uniform", lda=8, ldb=8, ldc=4)
    for row in oracle.gemm_f16(A, B, 3, 4, 5, C_in=C0):
        out.append("gemm_f16 3x4x5 accumulate " + " ".join(float(v).hex() for v in row))
    return out


if __name__ == "__main__":
    with open(os.path.join(HERE, "inputs_digest.txt"), "w") as f:
        f.write("\n".join(inputs_lines()) + "\n")
    with open(os.path.join(HERE, "oracle_tiny.txt"), "w") as f:
        f.write("\n".join(oracle_lines()) + "\n")
    print("written")
