"""Writes tests/golden/blob_digests.txt: SHA-256 of oracle-packed blobs of two fixed tiny cases.

Calls only the CPU oracle and the seeded input generators; run from the repository root:
    python tests/golden/make_golden.py
"""
import hashlib
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from paper_2012_00596_b200 import inputs  # noqa: E402

c = inputs.conv_case(N=1, H=4, W=4, C=16, K=16, Mb=8, Nb=8, keep=3, dtype="bf16", seed=71)
l = inputs.linear_case(M=1, I=32, O=32, Bo=16, Bi=16, keep_rows=4, keep_cols=5, dtype="bf16", seed=72)
with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "blob_digests.txt"), "w") as f:
    f.write("# sha256 of oracle.pack_bp / oracle.pack_bb output (format: module docstring of oracle/packers.py)\n")
    f.write("bp_8x8_bf16 %s\n" % hashlib.sha256(oracle.pack_bp(c.w, c.tap_mask, 8, 8, "bf16").tobytes()).hexdigest())
    f.write("bb_16x16_bf16 %s\n" % hashlib.sha256(oracle.pack_bb(l.w, l.row_keep, l.col_keep, 16, 16, "bf16").tobytes()).hexdigest())
