"""Comparison helpers shared by the GPU parity tests."""
import numpy as np

from paper_2408_00264_b200 import workloads as W

ATTN_MAX_ABS = 2e-2      # stated tolerance of the verify step: bf16 output, fp32 accumulation
ATTN_MAX_REL = 1e-2


def attn_errors(got_bits: np.ndarray, ref: np.ndarray):
    """got_bits [..., D] bf16 bits, ref [..., D] float64.  Returns (max abs error, max relative
    error).  The relative error is taken per output row (one (sequence, node, head) vector):
    max|got - ref| / max|ref|.  Probabilities enter the P.V product as bf16, which perturbs every
    output element by an amount proportional to the row's scale, not to the element itself, so an
    element-wise ratio is unbounded for elements that happen to be near zero; the row-normalised
    ratio is the one the arithmetic bounds (about 2^-8 from the two bf16 roundings)."""
    got = W.bf16_bits_to_f64(got_bits)
    err = np.abs(got - ref)
    row = np.abs(ref).max(axis=-1)
    rel = err.max(axis=-1) / np.maximum(row, 1e-30)
    return float(err.max()), float(rel.max())


def assert_attn_close(got_bits, ref, what=""):
    assert np.isfinite(W.bf16_bits_to_f64(got_bits)).all(), what
    a, r = attn_errors(got_bits, ref)
    assert a <= ATTN_MAX_ABS and r <= ATTN_MAX_REL, "%s max-abs %.3e max-rel %.3e" % (what, a, r)


def log_parity(workload, **figures):
    """Appends one line of observed parity figures to the file named by CLV_PARITY_LOG (if set)."""
    import json
    import os
    path = os.environ.get("CLV_PARITY_LOG")
    if not path:
        return
    os.makedirs(os.path.dirname(os.path.abspath(path)), exist_ok=True)
    with open(path, "a") as f:
        f.write(json.dumps(dict(workload=workload, **figures)) + "\n")
