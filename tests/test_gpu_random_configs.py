"""Seeded random configurations through the CUDA library and the CPU oracle.

Every case draws the replica count, the stage sizes (ragged, from one coordinate to a few
chunks), p, tau, the averaging interval, the look-ahead delays, the optimizer, the staleness
estimate, the exchange precision, the snapshot storage and the kernel flag, steps both sides
on the same seeded inputs and compares the whole state bit for bit: whichever kernel, form
and ring mode the library picks for the draw has to give the oracle's numbers.  The draws
are reproducible (one generator per case number); ASYNCMESH_RANDOM_CASES raises their
number."""
import os

import numpy as np
import pytest

from tests.test_gpu_parity import run_case

pytestmark = pytest.mark.gpu

N_CASES = int(os.environ.get("ASYNCMESH_RANDOM_CASES", "256"))
SIZES = [1, 3, 4, 5, 31, 127, 128, 129, 255, 256, 257, 1023, 1024, 1025, 2047, 2049, 3000, 4099, 5000, 9000,
         33000, 70001]


def draw(case):
    rng = np.random.default_rng(0xA5F0 + case)
    from paper_2601_22442_b200 import binding
    R = int(rng.choice([1, 2, 3, 4, 4, 4, 5, 6, 7, 8, 8, 8, 9, 12, 16]))
    S = int(rng.integers(1, 5))
    numel = [int(rng.choice(SIZES)) for _ in range(S)]
    p = float(rng.choice([0.0, 0.01, 0.05, 0.05, 0.1, 0.2, 0.3, 0.5, 0.8, 1.0]))
    K = int(rng.choice([1, 1, 1, 2, 3]))
    tau = K * int(rng.choice([0, 1, 1, 2, 3]))
    kw = dict(avg_interval=K, delays=[int(rng.integers(0, 4)) for _ in range(S)])
    kw["optimizer"] = str(rng.choice(["adamw", "adamw", "nadamw"]))
    kw["correction"] = str(rng.choice(["ema", "ema", "ema", "eager"]))
    kw["exchange"] = str(rng.choice(["fp32", "fp32", "bf16", "fp8"]))
    flag = int(rng.choice([0, 0, 0, binding.FLAG_DIRECT_KERNEL, binding.FLAG_PIPELINED_KERNEL,
                           binding.FLAG_OWNER_KERNEL, binding.FLAG_DENSE_RING]))
    if kw["exchange"] != "fp32" and tau > 0 and rng.random() < 0.3:
        kw["snapshot"] = "as-exchanged"      # implies the dense ring and the direct kernel
        flag = 0
    if rng.random() < 0.2:
        flag |= binding.FLAG_TRACK_CONSENSUS
    if rng.random() < 0.15:
        flag |= binding.FLAG_KEEP_PREVIOUS
    kw["flags"] = flag
    kw["same_init"] = bool(rng.random() < 0.5)
    lam = float(rng.choice([0.0, 0.3, 0.9, 1.0]))
    steps = 2 * tau + int(rng.integers(2, 6))
    return R, numel, p, tau, lam, steps, kw


@pytest.mark.parametrize("case", range(N_CASES))
def test_random_configuration(case):
    R, numel, p, tau, lam, steps, kw = draw(case)
    o, g = run_case(R, numel, p, tau, lam, steps, check_masks=(1, steps), **kw)
    for s in range(len(numel)):
        ce_o, ce_g = o.consensus_error(s), g.consensus_error(s)
        assert abs(ce_o - ce_g) <= 1e-9 * max(ce_o, 1e-30), (s, ce_o, ce_g)
