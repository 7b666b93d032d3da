"""GPU parity on values outside the comfortable range of the seeded inputs.

Weights and gradients are built by hand: subnormal, zero (both signs), tiny, huge,
infinite and NaN values, gradients that vanish after the moments have filled, moments
that never fill.  The CUDA library must agree with the CPU oracle bit for bit on every
number and on where the NaNs are (NaN payloads are not compared).

What these cases would catch:
  * flush-to-zero arithmetic (-ftz=true): the subnormal gradients 1e-40 leave subnormal
    first moments, which would read 0 on the device -> the `m` comparison fails;
  * an approximate division or square root: ordinary values then differ in the last bit
    -> the `w` comparison fails on the first step;
  * a straight-line division / square root used outside its operand range: zero or
    subnormal second moments (g = 0, 1e-30, 1e-40), overflowing squares (g = 1e25, 3e38)
    and infinities must take the toolkit's routines -> `w` or `look` would show a NaN or
    a wrong value where the oracle has 0, Inf or a finite number;
  * a replica mean that treats NaN or Inf specially -> `w` of the other replicas."""
import numpy as np
import pytest
import torch

import oracle
from tests.util import HP, STATE_NAMES

pytestmark = pytest.mark.gpu

SPECIAL_G = np.array([0.0, -0.0, 1e-40, -1e-40, 1.4e-45, 1e-30, -1e-30, 1e-20, 3e-19, 1e-3, -7e-4,
                      1.0, 1e18, -1e18, 1e25, 3e38, -3e38, np.inf, -np.inf, np.nan], dtype=np.float32)
TINY_G = np.array([1e-40, -1e-40, 1.4e-45, 0.0, 1e-30, -1e-30, 3e-39], dtype=np.float32)
SPECIAL_W = np.array([0.0, -0.0, 1e-40, -1e-40, 0.02, -0.02, 1.0, 500.0, -1000.0, 1e30, 3e38, -3e38],
                     dtype=np.float32)


def am():
    import paper_2601_22442_b200 as pkg
    return pkg


def build_inputs(R, n, steps, seed):
    """w0 [R][n] and grads [steps][R][n]: every coordinate walks through the special
    values in an order of its own; a third of the coordinates see ordinary gradients
    first and exact zeros afterwards (g = 0 with m != 0), a sixth never see anything but
    zeros (m = v = 0 throughout), a sixth only subnormal and tiny values (subnormal m, v = 0)."""
    rng = np.random.default_rng(seed)
    w0 = SPECIAL_W[rng.integers(0, SPECIAL_W.size, size=(R, n))]
    w0[:, ::3] = (0.02 * rng.standard_normal((R, (n + 2) // 3))).astype(np.float32)
    grads = []
    for t in range(steps):
        g = SPECIAL_G[rng.integers(0, SPECIAL_G.size, size=(R, n))]
        ordinary = (1e-3 * rng.standard_normal((R, n))).astype(np.float32)
        sign = np.where((np.arange(n) + t) % 2 == 0, 1.0, -1.0).astype(np.float32)   # alternating signs
        g[:, 1::3] = (np.abs(ordinary) * sign)[:, 1::3] if t < 2 else 0.0
        g[:, 5::6] = 0.0
        g[:, 2::6] = TINY_G[rng.integers(0, TINY_G.size, size=(R, len(range(2, n, 6))))]
        if R > 1:       # NaN and Inf only ever in replica 0: the mean must carry them to the others
            bad = ~np.isfinite(g[1:])
            g[1:][bad] = ordinary[1:][bad]
        grads.append(np.ascontiguousarray(g))
    return np.ascontiguousarray(w0), grads


def same_bits(a, b, what):
    a = np.ascontiguousarray(a, dtype=np.float32)
    b = np.ascontiguousarray(b, dtype=np.float32)
    na, nb = np.isnan(a), np.isnan(b)
    assert np.array_equal(na, nb), (what, "NaN in different places", int((na != nb).sum()))
    ua, ub = a.view(np.uint32)[~na], b.view(np.uint32)[~nb]
    bad = np.nonzero(ua != ub)[0]
    assert bad.size == 0, (what, "differs in %d values, first at %d: %r vs %r"
                           % (bad.size, bad[0], a[~na][bad[0]], b[~nb][bad[0]]))


def run(R, n, p, tau, flags, exchange="fp32", steps=7, seed=0, optimizer="adamw", snapshot="own-fp32"):
    numel = [n, n // 2 + 3]       # two stages: look-ahead delays 1 and 0
    xflag = {"fp32": 0, "bf16": 16, "fp8": 64}[exchange]
    o = oracle.Oracle(R, numel, p=p, tau=tau, ema_beta=0.9, seed=11, exchange=exchange, optimizer=optimizer,
                      snapshot=snapshot, **HP)
    flags |= {"own-fp32": 0, "as-exchanged": 1024}[snapshot]
    g = am().AsyncMesh(R, numel, p=p, tau=tau, ema_beta=0.9, seed=11, flags=flags | xflag, optimizer=optimizer, **HP)
    inputs = [build_inputs(R, m, steps, seed + s) for s, m in enumerate(numel)]
    for s in range(2):
        for i in range(R):
            o.init_params(s, inputs[s][0][i], replica=i)
            g.init_params(s, inputs[s][0][i], replica=i)
    bufs = g.empty_grads()
    for t in range(steps):
        for s, m in enumerate(numel):
            bufs[s][:, :m].copy_(torch.from_numpy(inputs[s][1][t]))
        o.step([inputs[s][1][t] for s in range(2)])
        g.step(bufs)
        if t == 0:      # the first step alone already pins division and square root
            same_bits(o.get(0, "w"), g.get(0, "w"), ("w after one step", R, p, tau, flags))
    g.status()
    for s in range(2):
        for name in STATE_NAMES:
            a, b = o.get(s, name), g.get(s, name)
            if name == "d" and tau == 0:
                # Synchronous averaging (Eq. "sparta") has no staleness term and the library never
                # touches d then.  The oracle applies Eq. "ema" literally, whose sample
                # w^ - w^ is 0 for every finite iterate but NaN for a NaN one: d is compared
                # where the oracle's iterate is a number, and must be 0 there.
                finite = ~np.isnan(o.get(s, "w"))
                assert not b.any()
                a, b = a[finite], b[finite]
            same_bits(a, b, (s, name, R, p, tau, flags, exchange))
    assert np.isnan(o.get(0, "w")).any() and np.isinf(o.get(0, "v")).any()   # the cases did occur
    assert (o.get(0, "m") != 0).any() and (np.abs(o.get(0, "m")[o.get(0, "m") != 0]) < 1.2e-38).any()


def flags_of(name):
    from paper_2601_22442_b200 import binding
    return {"default": 0, "direct": binding.FLAG_DIRECT_KERNEL, "pipelined": binding.FLAG_PIPELINED_KERNEL,
            "owner": binding.FLAG_OWNER_KERNEL, "dense": binding.FLAG_DENSE_RING}[name]


@pytest.mark.parametrize("kernel", ["default", "direct", "pipelined", "owner", "dense"])
@pytest.mark.parametrize("R", [1, 4, 8])
@pytest.mark.parametrize("p", [0.05, 1.0])
def test_edge_values_delayed_averaging(kernel, R, p):
    run(R, 3 * 1024 + 41, p, 2, flags_of(kernel))


@pytest.mark.parametrize("kernel", ["default", "direct", "pipelined", "owner"])
@pytest.mark.parametrize("R", [1, 4, 8])
@pytest.mark.parametrize("p", [0.05, 1.0])
def test_edge_values_synchronous_averaging(kernel, R, p):
    run(R, 2 * 1024 + 7, p, 0, flags_of(kernel), steps=4)


@pytest.mark.parametrize("kernel", ["default", "direct", "pipelined", "dense"])
@pytest.mark.parametrize("R", [4, 8])
def test_edge_values_with_the_8_bit_exchange(kernel, R):
    # weights beyond the largest E4M3 value (448) clamp in the exchange; NaN stays NaN
    run(R, 2 * 1024 + 7, 0.3, 2, flags_of(kernel), exchange="fp8")
    run(R, 1024 + 7, 0.3, 0, flags_of(kernel) & ~32, exchange="bf16", steps=4)


@pytest.mark.parametrize("exchange", ["bf16", "fp8"])
@pytest.mark.parametrize("R", [1, 4, 8])
def test_edge_values_with_the_ring_kept_as_exchanged(exchange, R):
    # infinities, NaN, subnormals and values beyond 448 pass through the 2- and 1-byte ring slots
    run(R, 2 * 1024 + 7, 0.5, 2, 0, exchange=exchange, snapshot="as-exchanged")
    run(R, 1024 + 7, 1.0, 1, 0, exchange=exchange, snapshot="as-exchanged", steps=4)


def test_edge_values_nadamw():
    run(4, 2 * 1024 + 7, 0.3, 2, 0, optimizer="nadamw")                          # owner kernel, NAdamW form
    run(4, 2 * 1024 + 7, 0.3, 2, flags_of("pipelined"), optimizer="nadamw")      # pipelined kernel, general form
    run(4, 2 * 1024 + 7, 0.3, 0, 0, optimizer="nadamw", steps=4)
    run(8, 2 * 1024 + 7, 0.3, 2, 0, optimizer="nadamw")


@pytest.mark.parametrize("case", range(48))
def test_edge_values_random_configuration(case):
    # the hand-built special values through whatever kernel, form and ring mode a seeded draw selects
    rng = np.random.default_rng(0xED6E + case)
    R = int(rng.choice([1, 2, 3, 4, 4, 5, 6, 8, 8, 12]))
    n = int(rng.choice([1024 + 7, 2 * 1024 + 41, 3 * 1024 + 5]))
    p = float(rng.choice([0.05, 0.2, 0.5, 1.0]))
    tau = int(rng.choice([0, 1, 2, 3]))
    exchange = str(rng.choice(["fp32", "fp32", "bf16", "fp8"]))
    snapshot = "as-exchanged" if exchange != "fp32" and tau > 0 and rng.random() < 0.4 else "own-fp32"
    kernel = str(rng.choice(["default", "default", "direct", "pipelined", "owner"]))
    flags = 0 if snapshot == "as-exchanged" else flags_of(kernel)
    optimizer = str(rng.choice(["adamw", "adamw", "nadamw"]))
    run(R, n, p, tau, flags, exchange=exchange, steps=int(rng.integers(4, 8)), seed=case, optimizer=optimizer,
        snapshot=snapshot)
