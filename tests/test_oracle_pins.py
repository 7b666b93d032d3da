"""Pins for the CPU oracle: every part of it is held to something other than
itself -- published vectors, a library optimizer, closed forms, the reductions
between the paper's equations, Lemma 1, and a brute-force trace."""
import os

import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from tests import bruteforce

HP = dict(lr=3e-4, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)
GOLD = os.path.join(os.path.dirname(__file__), "golden")


def relerr(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    den = np.maximum(np.abs(a), np.abs(b))
    with np.errstate(invalid="ignore", divide="ignore"):
        e = np.where(den > 0, np.abs(a - b) / den, 0.0)
    return float(e.max()) if e.size else 0.0


def rand_setup(R, N, steps, seed=7, stage=0, same_init=True):
    w0 = si.init_weights_host(seed, stage, 0, N)
    grads = [si.grads_host(seed + 1, t, stage, R, 0, N) for t in range(1, steps + 1)]
    return w0, grads


# ---- P0: Philox and the threshold -------------------------------------------

def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLD, "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        x = [int(h, 16) for h in r]
        assert oracle.philox4x32_10(x[0:4], x[4:6]) == tuple(x[6:10])
        assert tuple(bruteforce.philox(x[0:4], x[4:6])) == tuple(x[6:10])


def test_philox_matches_python_integers_on_random_inputs():
    rng = np.random.default_rng(0)
    for _ in range(200):
        c = [int(x) for x in rng.integers(0, 1 << 32, 4)]
        k = [int(x) for x in rng.integers(0, 1 << 32, 2)]
        assert oracle.philox4x32_10(c, k) == tuple(bruteforce.philox(c, k))


def test_threshold_edges():
    # floor(p * 2^32) in double; the fp32 value of 0.05 would give another T
    assert oracle.threshold(0.0) == 0
    assert oracle.threshold(1.0) == 1 << 32
    assert oracle.threshold(0.05) == 214748364
    assert oracle.threshold(2.0 ** -32) == 1
    assert oracle.threshold(0.5) == 1 << 31


def test_subset_is_per_stage_per_step_and_shared_by_replicas():
    o = oracle.Oracle(3, [4099, 4099], p=0.3, tau=0, ema_beta=0.5)
    a, b = o.subset_mask(0, 5), o.subset_mask(1, 5)
    c = o.subset_mask(0, 6)
    assert (a != b).any() and (a != c).any()
    assert (a == o.subset_mask(0, 5)).all()
    for mu in (0, 1, 2, 3, 4, 4098):
        assert a[mu] == bruteforce.in_subset(o.seed, 0.3, 0, 5, mu)
        assert a[mu] == oracle.selected(o.seed, 0.3, 0, 5, mu)


@pytest.mark.parametrize("p", [0.01, 0.05, 0.25])
def test_selection_rate(p):
    N = 1 << 22
    o = oracle.Oracle(1, [N], p=p, tau=0, ema_beta=0.5)
    k = int(o.subset_mask(0, 3).sum())
    sigma = np.sqrt(N * p * (1 - p))
    assert abs(k - N * p) < 4 * sigma
    # the four output words of one block are all used: rate holds per lane
    m = o.subset_mask(0, 3).reshape(-1, 4).sum(0)
    assert (np.abs(m - N / 4 * p) < 5 * np.sqrt(N / 4 * p * (1 - p))).all()


def test_p_zero_and_one():
    o0 = oracle.Oracle(1, [1000], p=0.0, tau=0, ema_beta=0.5)
    o1 = oracle.Oracle(1, [1000], p=1.0, tau=0, ema_beta=0.5)
    assert not o0.subset_mask(0, 1).any()
    assert o1.subset_mask(0, 1).all()


# ---- P1: the optimizer --------------------------------------------------------

def torch_adamw_run(w0, grads_per_step, dtype):
    """grads_per_step[t] is one replica's gradient vector."""
    p = torch.nn.Parameter(torch.tensor(w0, dtype=dtype))
    opt = torch.optim.AdamW([p], lr=HP["lr"], betas=(HP["beta1"], HP["beta2"]),
                            eps=HP["eps"], weight_decay=HP["weight_decay"])
    for g in grads_per_step:
        p.grad = torch.tensor(g, dtype=dtype)
        opt.step()
    st = opt.state[p]
    return (p.detach().numpy(), st["exp_avg"].numpy(), st["exp_avg_sq"].numpy())


def test_adamw_against_torch_library():
    R, N, T = 2, 1 << 14, 100
    w0, grads = rand_setup(R, N, T)
    o = oracle.Oracle(R, [N], p=0.0, tau=0, ema_beta=0.9, lookahead_delay=[0], **HP)
    o.init_params(0, w0)
    for g in grads:
        o.step([g])
    for i in range(R):
        w64, m64, v64 = torch_adamw_run(w0, [g[i] for g in grads], torch.float64)
        # fp32 rounding of ~10 operations per step in contracting recursions:
        # a few 1e-7 of the gradient scale (1e-3) on m, whose signed terms
        # cancel, a few 1e-7 relative on v, whose terms are all positive, and
        # far less on w (one update is 1e-2 of |w|)
        assert np.abs(o.row(0, "m", i) - m64).max() < 1e-6 * 1e-3
        assert relerr(o.row(0, "v", i), v64) < 2e-6
        assert np.abs(o.row(0, "w", i) - w64).max() < 1e-7
        w32, _, _ = torch_adamw_run(w0, [g[i] for g in grads], torch.float32)
        # the fp32 library run takes its own rounding walk (other operation
        # order): two walks of ~2 roundings a step at |w| <= 0.1
        assert np.abs(o.row(0, "w", i) - w32).max() < 4e-7
    assert not o.get(0, "d").any()


def test_adamw_constant_gradient_closed_form():
    # constant g, no decay: m^ = g and v^ = g^2 at every step, so every update
    # is -lr * g / (|g| + eps)
    N, T = 257, 30
    g = np.linspace(-2.0, 2.0, N).astype(np.float32)
    g[N // 2] = 0.5
    w0 = np.zeros(N, dtype=np.float32)
    hp = dict(HP, weight_decay=0.0)
    o = oracle.Oracle(1, [N], p=0.0, tau=0, ema_beta=0.9, lookahead_delay=[0], **hp)
    o.init_params(0, w0)
    for _ in range(T):
        o.step([g[None, :]])
    g64 = g.astype(np.float64)
    expect = -T * HP["lr"] * g64 / (np.abs(g64) + HP["eps"])
    assert np.abs(o.row(0, "w", 0) - expect).max() < 5e-6 * HP["lr"] * T


def test_nadamw_against_torch_library():
    # the paper's optimizer for asynchronous pipelines: NAdam with decoupled decay,
    # momentum 0.99
    R, N, T = 2, 1 << 13, 60
    w0, grads = rand_setup(R, N, T)
    hp = dict(HP, beta1=0.99)
    o = oracle.Oracle(R, [N], p=0.0, tau=0, ema_beta=0.9, lookahead_delay=[0],
                      optimizer="nadamw", **hp)
    o.init_params(0, w0)
    for g in grads:
        o.step([g])
    for i in range(R):
        q = torch.nn.Parameter(torch.tensor(w0, dtype=torch.float64))
        opt = torch.optim.NAdam([q], lr=hp["lr"], betas=(hp["beta1"], hp["beta2"]), eps=hp["eps"],
                                weight_decay=hp["weight_decay"], momentum_decay=4e-3,
                                decoupled_weight_decay=True)
        for g in grads:
            q.grad = torch.tensor(g[i], dtype=torch.float64)
            opt.step()
        st = opt.state[q]
        assert np.abs(o.row(0, "w", i) - q.detach().numpy()).max() < 2e-7
        assert np.abs(o.row(0, "m", i) - st["exp_avg"].numpy()).max() < 1e-9
        assert relerr(o.row(0, "v", i), st["exp_avg_sq"].numpy()) < 2e-6
    # and it is not AdamW
    a = oracle.Oracle(R, [N], p=0.0, tau=0, ema_beta=0.9, lookahead_delay=[0], **hp)
    a.init_params(0, w0)
    for g in grads:
        a.step([g])
    assert np.abs(a.row(0, "w", 0) - o.row(0, "w", 0)).max() > 1e-5


# ---- P2: p = 1, tau = 0 is "average everything every step" --------------------

def test_full_sync_averaging_against_torch():
    R, N, T = 4, 4096, 20
    w0, grads = rand_setup(R, N, T)
    o = oracle.Oracle(R, [N], p=1.0, tau=0, ema_beta=0.9, **HP)
    o.init_params(0, w0)
    ps = [torch.nn.Parameter(torch.tensor(w0, dtype=torch.float64)) for _ in range(R)]
    opts = [torch.optim.AdamW([q], lr=HP["lr"], betas=(HP["beta1"], HP["beta2"]),
                              eps=HP["eps"], weight_decay=HP["weight_decay"]) for q in ps]
    for g in grads:
        o.step([g])
        for i in range(R):
            ps[i].grad = torch.tensor(g[i], dtype=torch.float64)
            opts[i].step()
        mean = torch.stack([q.detach() for q in ps]).mean(0)
        for q in ps:
            q.data.copy_(mean)
        W = o.get(0, "w")
        assert (W == W[0]).all()           # replicas identical after every step
        assert np.abs(W[0] - mean.numpy()).max() < 1e-7
    assert not o.get(0, "d").any()


# ---- P3 / P4 / P5: reductions between the paper's equations -------------------

def seq_mean_f32(A):
    acc = A[0].astype(np.float32)
    for i in range(1, A.shape[0]):
        acc = (acc + A[i]).astype(np.float32)
    return (acc / np.float32(A.shape[0])).astype(np.float32)


@pytest.mark.parametrize("tau", [1, 3])
def test_lambda_zero_is_plain_delayed_averaging(tau):
    R, N, T = 3, 2051, 12
    w0, grads = rand_setup(R, N, T)
    o = oracle.Oracle(R, [N], p=0.3, tau=tau, ema_beta=0.0, **HP)
    o.init_params(0, w0)
    hist = {}
    for t, g in enumerate(grads, 1):
        o.step([g])
        hist[t] = o.get(0, "what")
        W = o.get(0, "w")
        if t > tau:
            sel = o.subset_mask(0, t - tau)
            assert 0 < sel.sum() < N
            wbar = seq_mean_f32(hist[t - tau])
            for i in range(R):
                assert (W[i][sel] == wbar[sel]).all()            # old average
                assert (W[i][~sel] == hist[t][i][~sel]).all()    # local value
        else:
            assert (W == hist[t]).all()
    assert not o.get(0, "d").any()


def test_lambda_one_is_raw_difference():
    R, N, T, tau = 2, 1027, 9, 2
    w0, grads = rand_setup(R, N, T)
    o = oracle.Oracle(R, [N], p=0.4, tau=tau, ema_beta=1.0, **HP)
    o.init_params(0, w0)
    hist = {}
    dref = np.zeros((R, N), dtype=np.float32)
    for t, g in enumerate(grads, 1):
        o.step([g])
        hist[t] = o.get(0, "what")
        if t > tau:
            sel = o.subset_mask(0, t - tau)
            diff = (hist[t] - hist[t - tau]).astype(np.float32)
            dref[:, sel] = diff[:, sel]
            wbar = seq_mean_f32(hist[t - tau])
            W = o.get(0, "w")
            assert (W[:, sel] == (wbar[sel] + dref[:, sel]).astype(np.float32)).all()
        assert (o.get(0, "d") == dref).all()


@pytest.mark.parametrize("lam", [0.0, 0.5, 0.9, 1.0])
def test_tau_zero_is_synchronous_sparse_averaging(lam):
    R, N, T = 4, 3001, 8
    w0, grads = rand_setup(R, N, T)
    o = oracle.Oracle(R, [N], p=0.25, tau=0, ema_beta=lam, **HP)
    o.init_params(0, w0)
    for t, g in enumerate(grads, 1):
        o.step([g])
        what, W = o.get(0, "what"), o.get(0, "w")
        sel = o.subset_mask(0, t)
        wbar = seq_mean_f32(what)
        assert (W[:, sel] == wbar[sel]).all()
        assert (W[:, ~sel] == what[:, ~sel]).all()
    assert not o.get(0, "d").any()


# ---- P6: mean invariance and Lemma 1 -------------------------------------------

def test_mean_invariance_and_lemma1_shrink_factor():
    R, N, p = 4, 1 << 20, 0.05
    o = oracle.Oracle(R, [N], p=p, tau=0, ema_beta=0.9, **HP)
    for i in range(R):   # replicas deliberately apart: different starting points
        o.init_params(0, si.normal_host(si.stream_key(3, si.KIND_INIT, 0, 0, i), 0, N, 0.02),
                      replica=i)
    g = si.grads_host(11, 1, 0, R, 0, N)
    o.step([g])
    what = o.get(0, "what").astype(np.float64)
    W = o.get(0, "w").astype(np.float64)
    # averaging replaces values by their mean: the replica mean is unchanged
    assert np.abs(W.mean(0) - what.mean(0)).max() < 2 * np.finfo(np.float32).eps * 0.1
    before = ((what - what.mean(0)) ** 2).sum(0)       # per coordinate
    after = ((W - W.mean(0)) ** 2).sum(0)
    # Lemma 1: E[after] = (1 - p) E[before]; the only randomness is the subset
    expect = (1 - p) * before.sum()
    sigma = np.sqrt(p * (1 - p) * (before ** 2).sum())
    assert abs(after.sum() - expect) < 4 * sigma
    assert abs(o.consensus_error(0) - after.sum()) < 1e-9 * after.sum()
    sel = o.subset_mask(0, 1)
    assert after[sel].max() < 1e-12 and (after[~sel] == before[~sel]).all()


# ---- P7: look-ahead --------------------------------------------------------------

def test_lookahead_zero_delay_is_identity():
    R, N, T = 2, 515, 5
    w0, grads = rand_setup(R, N, T)
    o = oracle.Oracle(R, [N, N], p=0.2, tau=1, ema_beta=0.9,
                      lookahead_delay=[0, 0], **HP)
    o.init_params(0, w0); o.init_params(1, w0)
    assert (o.get(0, "look") == o.get(0, "w")).all()   # before any step
    for g in grads:
        o.step([g, g])
        assert (o.get(0, "look") == o.get(0, "w")).all()
        assert (o.get(1, "look") == o.get(1, "w")).all()


def test_lookahead_zero_delay_is_identity_on_infinite_and_signed_zero_weights():
    # "the look-ahead with zero delay returns the current weights": bit for bit, also where
    # w + 0 * (w - w_prev) would not (0 * (Inf - Inf) is NaN; -0 + 0 is +0)
    w0 = np.array([np.inf, -np.inf, -0.0, 0.0, 3e38, -3e38, 1.0, np.nan], dtype=np.float32)
    hp = dict(HP, weight_decay=0.0)
    o = oracle.Oracle(1, [w0.size, w0.size], p=0.0, tau=1, ema_beta=0.9, lookahead_delay=[0, 2], **hp)
    o.init_params(0, w0); o.init_params(1, w0)
    g = np.zeros((1, w0.size), dtype=np.float32)
    for _ in range(3):
        o.step([g, g])
        w, look = o.get(0, "w"), o.get(0, "look")
        assert np.array_equal(w.view(np.uint32), look.view(np.uint32))
        assert np.array_equal(o.lookahead(0, 0).view(np.uint32), w.view(np.uint32))
        assert np.array_equal(o.lookahead(1, 0).view(np.uint32), o.get(1, "w").view(np.uint32))
    # before any step w^{-1} = w^0: with a delay the formula applies, and Inf - Inf is NaN
    o3 = oracle.Oracle(1, [w0.size], p=0.0, tau=1, ema_beta=0.9, lookahead_delay=[2], **hp)
    o3.init_params(0, w0)
    assert np.isnan(o3.lookahead(0, 2)[0, 0]) and o3.lookahead(0, 0)[0, 0] == np.inf
    assert np.signbit(o3.lookahead(0, 0)[0, 2]) and not np.signbit(o3.lookahead(0, 2)[0, 2])


def test_lookahead_default_delay_and_constant_velocity():
    # default delay is S-1-stage; with a constant update direction the
    # extrapolation by k steps lands on the weights k steps later
    N, S, T = 129, 4, 12
    g = np.linspace(-1.0, 1.0, N).astype(np.float32)
    g[np.abs(g) < 1e-3] = 0.25
    hp = dict(HP, weight_decay=0.0)
    o = oracle.Oracle(1, [N] * S, p=0.0, tau=0, ema_beta=0.9, **hp)
    for s in range(S):
        o.init_params(s, np.zeros(N, dtype=np.float32))
    looks, ws = {}, {}
    for t in range(1, T + 1):
        o.step([g[None, :]] * S)
        looks[t] = [o.row(s, "look", 0) for s in range(S)]
        ws[t] = o.row(0, "w", 0)
    for s in range(S):
        k = S - 1 - s
        t = 5
        assert np.abs(looks[t][s] - ws[t + k]).max() < 1e-6 * np.abs(ws[t + k]).max()
    # and the definition itself, from what the oracle exposes
    s = 1
    w, wp = o.row(s, "w", 0), o.row(s, "wprev", 0)
    assert (o.row(s, "look", 0) == (w + np.float32(2) * (w - wp)).astype(np.float32)).all()


def test_lookahead_for_any_delay():
    # delay 0 is the weights, the configured delay is what the step wrote, and under a
    # constant update direction delay k lands on the weights k steps later
    N, T = 129, 14
    g = np.linspace(-1.0, 1.0, N).astype(np.float32)
    g[np.abs(g) < 1e-3] = 0.25
    o = oracle.Oracle(1, [N], p=0.0, tau=0, ema_beta=0.9, lookahead_delay=[3],
                      **dict(HP, weight_decay=0.0))
    o.init_params(0, np.zeros(N, dtype=np.float32))
    assert (o.lookahead(0, 7) == o.get(0, "w")).all()        # before any step: w^{-1} = w^0
    snap, ws = {}, {}
    for t in range(1, T + 1):
        o.step([g[None, :]])
        ws[t] = o.get(0, "w")
        assert (o.lookahead(0, 0) == ws[t]).all()
        assert (o.lookahead(0, 3) == o.get(0, "look")).all()
        if t == 5:
            snap = {k: o.lookahead(0, k) for k in (1, 2, 6, 9)}
    for k, look in snap.items():
        assert np.abs(look - ws[5 + k]).max() < 1e-6 * np.abs(ws[5 + k]).max()
    # a brute-force trace agrees with the oracle's own look at a delay both computed
    R, N2, seed = 2, 16, 0xABC
    w0, grads = rand_setup(R, N2, 4, seed=9)
    o2 = oracle.Oracle(R, [N2], p=0.5, tau=1, ema_beta=0.9, seed=seed, lookahead_delay=[1], **HP)
    o2.init_params(0, w0)
    tr = bruteforce.run(np.float32, R, N2, 0.5, 1, 0.9, HP["lr"], HP["beta1"], HP["beta2"], HP["eps"],
                        HP["weight_decay"], seed, 5, w0, grads)
    for t in range(4):
        o2.step([grads[t]])
        assert (o2.lookahead(0, 5).astype(np.float64) == tr[t]["look"]).all()


# ---- P8: brute-force trace --------------------------------------------------------

@pytest.mark.parametrize("tau,p,lam", [(2, 0.5, 0.9), (1, 0.3, 0.5), (0, 0.5, 0.9), (3, 1.0, 0.1)])
def test_bruteforce_trace(tau, p, lam):
    R, N, T, seed, delay = 2, 16, 7, 0xABCDEF0123, 3
    w0, grads = rand_setup(R, N, T, seed=5)
    o = oracle.Oracle(R, [N], p=p, tau=tau, ema_beta=lam, seed=seed,
                      lookahead_delay=[delay], **HP)
    o.init_params(0, w0)
    args = (R, N, p, tau, lam, HP["lr"], HP["beta1"], HP["beta2"], HP["eps"],
            HP["weight_decay"], seed, delay, w0, grads)
    t32 = bruteforce.run(np.float32, *args)
    t64 = bruteforce.run(np.float64, *args)
    touched = 0
    for t in range(1, T + 1):
        o.step([grads[t - 1]])
        assert sorted(np.nonzero(o.subset_mask(0, t))[0].tolist()) == t32[t - 1]["subset"]
        for name in ("w", "m", "v", "d", "look", "what"):
            got = o.get(0, name)
            assert (got.astype(np.float64) == t32[t - 1][name]).all(), (t, name)
            # against the float64 trace: sums of signed terms (m, the staleness
            # w^t - w^{t-tau}, the direction w^t - w^{t-1}) cancel, so those are
            # held to an absolute bound at the scale of their terms; v is a sum of
            # positive terms and is held to a relative one
            ref = t64[t - 1][name]
            if name == "v":
                assert relerr(got, ref) < 2e-6, (t, name)
            else:
                bound = {"m": 1e-9, "w": 3e-8, "what": 3e-8, "d": 5e-8, "look": 1e-7}[name]
                assert np.abs(got - ref).max() < bound, (t, name)
        touched += int(np.count_nonzero(o.get(0, "d")))
    if tau > 0:
        assert touched > 0


def test_bruteforce_trace_second_stage_uses_its_own_subset():
    R, N, T, seed = 2, 16, 4, 99
    w0, grads = rand_setup(R, N, T, seed=8)
    o = oracle.Oracle(R, [N, N], p=0.5, tau=1, ema_beta=0.9, seed=seed,
                      lookahead_delay=[1, 0], **HP)
    o.init_params(0, w0); o.init_params(1, w0)
    args = (R, N, 0.5, 1, 0.9, HP["lr"], HP["beta1"], HP["beta2"], HP["eps"],
            HP["weight_decay"], seed, 0, w0, grads)
    tr = bruteforce.run(np.float32, *args, stage=1)
    for t in range(1, T + 1):
        o.step([grads[t - 1], grads[t - 1]])
        assert (o.get(1, "w").astype(np.float64) == tr[t - 1]["w"]).all()
    assert (o.get(0, "w") != o.get(1, "w")).any()


@pytest.mark.parametrize("K,tau", [(2, 2), (3, 0), (2, 4), (4, 4)])
def test_bruteforce_trace_with_averaging_interval(K, tau):
    # averaging every K steps: the steps in between are purely local
    R, N, T, seed = 3, 16, 13, 0x77
    w0, grads = rand_setup(R, N, T, seed=21)
    o = oracle.Oracle(R, [N], p=0.5, tau=tau, ema_beta=0.7, seed=seed,
                      lookahead_delay=[2], avg_interval=K, **HP)
    o.init_params(0, w0)
    args = (R, N, 0.5, tau, 0.7, HP["lr"], HP["beta1"], HP["beta2"], HP["eps"],
            HP["weight_decay"], seed, 2, w0, grads)
    tr = bruteforce.run(np.float32, *args, interval=K)
    changed = 0
    for t in range(1, T + 1):
        o.step([grads[t - 1]])
        for name in ("w", "m", "v", "d", "look"):
            assert (o.get(0, name).astype(np.float64) == tr[t - 1][name]).all(), (t, name)
        same = (o.get(0, "w") == o.get(0, "what")).all()
        if t % K != 0 or t <= tau:
            assert same                      # a local step: nothing is averaged
        else:
            changed += int(not same)
    assert changed > 0
    with pytest.raises(ValueError):
        oracle.Oracle(R, [N], p=0.5, tau=3, ema_beta=0.7, avg_interval=2)


def test_bf16_rounding_against_the_tensor_library():
    rng = np.random.default_rng(5)
    xs = np.concatenate([
        rng.standard_normal(20000).astype(np.float32) * 0.02,
        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40, -1e-40,
                  1.0 + 2 ** -8, 1.0 + 3 * 2 ** -9], dtype=np.float32)])   # ties and edges
    ref = torch.tensor(xs).to(torch.bfloat16).to(torch.float32).numpy()
    got = np.array([oracle.exchanged(float(x)) for x in xs], dtype=np.float32)
    assert np.array_equal(got.view(np.uint32), ref.view(np.uint32))
    assert oracle.exchanged(0.1234567, "fp32") == float(np.float32(0.1234567))


@pytest.mark.parametrize("tau", [0, 2])
def test_bruteforce_trace_with_bf16_exchange(tau):
    # the average is formed from bfloat16-rounded snapshots, the staleness sample
    # from the replica's own unrounded value
    R, N, T, seed = 3, 16, 8, 0x99
    w0, grads = rand_setup(R, N, T, seed=31)
    o = oracle.Oracle(R, [N], p=0.5, tau=tau, ema_beta=0.6, seed=seed, lookahead_delay=[1],
                      exchange="bf16", **HP)
    ref = oracle.Oracle(R, [N], p=0.5, tau=tau, ema_beta=0.6, seed=seed, lookahead_delay=[1], **HP)
    o.init_params(0, w0); ref.init_params(0, w0)
    args = (R, N, 0.5, tau, 0.6, HP["lr"], HP["beta1"], HP["beta2"], HP["eps"],
            HP["weight_decay"], seed, 1, w0, grads)
    tr = bruteforce.run(np.float32, *args, wire="bf16")
    for t in range(1, T + 1):
        o.step([grads[t - 1]]); ref.step([grads[t - 1]])
        for name in ("w", "m", "v", "d", "look"):
            assert (o.get(0, name).astype(np.float64) == tr[t - 1][name]).all(), (t, name)
    diff = np.abs(o.get(0, "w") - ref.get(0, "w")).max()
    assert 0 < diff < 1e-3        # it matters, by about a bfloat16 ulp of |w| ~ 0.05


def e4m3_grid():
    """All finite non-negative E4M3 values from the format's definition: bias 7, three
    mantissa bits, subnormals at exponent field 0, top code of the top binade unused."""
    vals = []
    for e in range(16):
        for mant in range(8):
            if e == 15 and mant == 7:
                continue                      # the NaN code
            vals.append(mant / 8 * 2.0 ** -6 if e == 0 else (1 + mant / 8) * 2.0 ** (e - 7))
    return vals


def test_fp8_rounding_against_the_format_and_the_tensor_library():
    grid = e4m3_grid()
    assert grid[-1] == 448.0 and grid[1] == 2.0 ** -9 and len(grid) == 127
    for k, x in enumerate(grid):              # representable values are fixed points
        assert oracle.exchanged(x, "fp8") == x and oracle.exchanged(-x, "fp8") == -x
        if k + 1 < len(grid):                 # the midpoint goes to the even code
            mid = (x + grid[k + 1]) / 2
            want = x if k % 2 == 0 else grid[k + 1]
            assert oracle.exchanged(mid, "fp8") == want, (x, grid[k + 1])
            assert oracle.exchanged(float(np.nextafter(np.float32(mid), np.float32(1e9))), "fp8") == grid[k + 1]
            assert oracle.exchanged(float(np.nextafter(np.float32(mid), np.float32(0))), "fp8") == x
    assert oracle.exchanged(460.0, "fp8") == 448.0 and oracle.exchanged(-1e9, "fp8") == -448.0
    assert oracle.exchanged(2.0 ** -11, "fp8") == 0.0    # below half the smallest subnormal
    rng = np.random.default_rng(6)
    xs = (rng.standard_normal(20000) * np.exp(rng.standard_normal(20000) * 3)).astype(np.float32)
    xs = xs[np.abs(xs) <= 448]
    ref = torch.tensor(xs).to(torch.float8_e4m3fn).to(torch.float32).numpy()
    got = np.array([oracle.exchanged(float(x), "fp8") for x in xs], dtype=np.float32)
    assert np.array_equal(got.view(np.uint32), ref.view(np.uint32))


@pytest.mark.parametrize("tau", [0, 2])
def test_bruteforce_trace_with_fp8_exchange(tau):
    R, N, T, seed = 3, 16, 8, 0x9A
    w0, grads = rand_setup(R, N, T, seed=33)
    o = oracle.Oracle(R, [N], p=0.5, tau=tau, ema_beta=0.6, seed=seed, lookahead_delay=[1],
                      exchange="fp8", **HP)
    ref = oracle.Oracle(R, [N], p=0.5, tau=tau, ema_beta=0.6, seed=seed, lookahead_delay=[1], **HP)
    o.init_params(0, w0); ref.init_params(0, w0)
    args = (R, N, 0.5, tau, 0.6, HP["lr"], HP["beta1"], HP["beta2"], HP["eps"],
            HP["weight_decay"], seed, 1, w0, grads)
    tr = bruteforce.run(np.float32, *args, wire="fp8")
    for t in range(1, T + 1):
        o.step([grads[t - 1]]); ref.step([grads[t - 1]])
        for name in ("w", "m", "v", "d", "look"):
            assert (o.get(0, name).astype(np.float64) == tr[t - 1][name]).all(), (t, name)
    diff = np.abs(o.get(0, "w") - ref.get(0, "w")).max()
    assert 1e-4 < diff < 1e-2     # about an E4M3 step (2^-4 relative) of |w| ~ 0.05


@pytest.mark.parametrize("wire,lo,hi", [("bf16", 0.0, 1e-3), ("fp8", 1e-4, 2e-2)])
def test_bruteforce_trace_with_the_snapshot_kept_only_as_exchanged(wire, lo, hi):
    # second reading of the reduced-precision exchange: the staleness sample is taken
    # against the rounded snapshot, because nothing else was kept
    R, N, T, seed, tau = 3, 16, 9, 0x9B, 2
    w0, grads = rand_setup(R, N, T, seed=35)
    kw = dict(p=0.5, tau=tau, ema_beta=0.6, seed=seed, lookahead_delay=[1], exchange=wire, **HP)
    o = oracle.Oracle(R, [N], snapshot="as-exchanged", **kw)
    first = oracle.Oracle(R, [N], **kw)
    o.init_params(0, w0); first.init_params(0, w0)
    args = (R, N, 0.5, tau, 0.6, HP["lr"], HP["beta1"], HP["beta2"], HP["eps"],
            HP["weight_decay"], seed, 1, w0, grads)
    tr = bruteforce.run(np.float32, *args, wire=wire, keeps_own_copy=False)
    for t in range(1, T + 1):
        o.step([grads[t - 1]]); first.step([grads[t - 1]])
        for name in ("w", "m", "v", "d", "look"):
            assert (o.get(0, name).astype(np.float64) == tr[t - 1][name]).all(), (t, name)
    # the two readings differ in d (it now carries the rounding error of the snapshot) ...
    diff = np.abs(o.get(0, "d") - first.get(0, "d")).max()
    assert lo < diff < hi
    # ... and not at all while the exchange is exact
    kw["exchange"] = "fp32"
    a, b = oracle.Oracle(R, [N], snapshot="as-exchanged", **kw), oracle.Oracle(R, [N], **kw)
    a.init_params(0, w0); b.init_params(0, w0)
    for t in range(1, T + 1):
        a.step([grads[t - 1]]); b.step([grads[t - 1]])
    assert all(np.array_equal(a.get(0, n), b.get(0, n)) for n in ("w", "d", "look"))


def test_snapshot_kept_as_exchanged_closed_form_of_one_round():
    # One replica, p = 1, tau = 1, lambda = 1, no weight decay: at step 2 the average of
    # one replica is its rounded snapshot q(w^^1), the staleness estimate is
    # d = w^^2 - q(w^^1), so w^2 = q(w^^1) + (w^^2 - q(w^^1)), all in fp32; under the
    # first reading d = w^^2 - w^^1 and w^2 = q(w^^1) + (w^^2 - w^^1).
    N = 64
    rng = np.random.default_rng(77)
    w0 = (0.05 * rng.standard_normal(N)).astype(np.float32)
    g = [(1e-2 * rng.standard_normal((1, N))).astype(np.float32) for _ in range(2)]
    hp = dict(HP, weight_decay=0.0)
    for wire in ("bf16", "fp8"):
        q = lambda x: torch.tensor(x).to({"bf16": torch.bfloat16, "fp8": torch.float8_e4m3fn}[wire]).to(torch.float32).numpy()
        for snapshot in ("as-exchanged", "own-fp32"):
            o = oracle.Oracle(1, [N], p=1.0, tau=1, ema_beta=1.0, exchange=wire, snapshot=snapshot, **hp)
            o.init_params(0, w0)
            o.step([g[0]])
            wh1 = o.get(0, "what")[0].copy()
            o.step([g[1]])
            wh2 = o.get(0, "what")[0].copy()
            mine = q(wh1) if snapshot == "as-exchanged" else wh1
            d = (wh2 - mine).astype(np.float32)
            assert np.array_equal(o.get(0, "d")[0], d)
            assert np.array_equal(o.get(0, "w")[0], (q(wh1) + d).astype(np.float32))
            assert (q(wh1) != wh1).any()


# ---- eager staleness estimate (end of Section 3.2) --------------------------------

@pytest.mark.parametrize("p,tau,K", [(1.0, 2, 2), (1.0, 3, 3), (0.5, 2, 1)])
def test_eager_estimate_bruteforce_and_closed_form(p, tau, K):
    R, N, T, seed = 3, 16, 10, 0x51
    w0, grads = rand_setup(R, N, T, seed=41)
    o = oracle.Oracle(R, [N], p=p, tau=tau, ema_beta=0.3, seed=seed, lookahead_delay=[1],
                      avg_interval=K, correction="eager", **HP)
    o.init_params(0, w0)
    args = (R, N, p, tau, 0.3, HP["lr"], HP["beta1"], HP["beta2"], HP["eps"],
            HP["weight_decay"], seed, 1, w0, grads)
    tr = bruteforce.run(np.float32, *args, interval=K, correction="eager")
    hist = {}
    rounds = 0
    for t in range(1, T + 1):
        o.step([grads[t - 1]])
        hist[t] = o.get(0, "what")
        for name in ("w", "m", "v", "d", "look"):
            assert (o.get(0, name).astype(np.float64) == tr[t - 1][name]).all(), (t, name)
        if t % K == 0 and t > tau:
            # closed form in double: w_i = mean_k w^_k^{t-tau} + (w^_i^t - w^_i^{t-tau}) / R
            sel = o.subset_mask(0, t - tau)
            old, now = hist[t - tau].astype(np.float64), hist[t].astype(np.float64)
            want = old.mean(axis=0) + (now - old) / R
            got = o.get(0, "w").astype(np.float64)
            assert np.abs(got[:, sel] - want[:, sel]).max() < 3e-8
            assert (got[:, ~sel] == now[:, ~sel]).all()
            # the replica mean moves by 1/R of the mean progress made since t - tau
            assert np.abs(got[:, sel].mean(axis=0)
                          - (old.mean(axis=0) + (now.mean(axis=0) - old.mean(axis=0)) / R)[sel]).max() < 3e-8
            rounds += 1
    assert rounds > 0


def test_eager_estimate_ignores_lambda_and_differs_from_the_ema():
    R, N, T = 4, 64, 6
    w0, grads = rand_setup(R, N, T, seed=43)
    runs = {}
    for name, kw in {"eager_a": dict(correction="eager", ema_beta=0.1),
                     "eager_b": dict(correction="eager", ema_beta=0.9),
                     "ema": dict(correction="ema", ema_beta=0.9)}.items():
        o = oracle.Oracle(R, [N], p=1.0, tau=2, seed=3, avg_interval=2, **kw, **HP)
        o.init_params(0, w0)
        for t in range(T):
            o.step([grads[t]])
        runs[name] = o.get(0, "w")
    assert (runs["eager_a"] == runs["eager_b"]).all()
    assert (runs["eager_a"] != runs["ema"]).any()


# ---- spread of the staleness estimates across replicas ------------------------------

def test_ema_variance_against_numpy():
    R, N, T = 4, 256, 9
    w0, grads = rand_setup(R, N, T, seed=47)
    o = oracle.Oracle(R, [N], p=0.5, tau=2, ema_beta=0.5, seed=11, **HP)
    o.init_params(0, w0)
    assert o.ema_variance(0) == (0.0, 0.0)
    for t in range(T):
        o.step([grads[t]])
    var = o.get(0, "d").astype(np.float64).var(axis=0)      # population variance over replicas
    mean, mx = o.ema_variance(0)
    assert mx > 0 and abs(mean - var.mean()) <= 1e-12 * var.mean() and abs(mx - var.max()) <= 1e-12 * mx
    # identical replicas (same gradients everywhere): the estimates agree, variance 0
    o2 = oracle.Oracle(R, [N], p=0.5, tau=2, ema_beta=0.5, seed=11, **HP)
    o2.init_params(0, w0)
    for t in range(T):
        o2.step([np.repeat(grads[t][:1], R, axis=0)])
    assert np.abs(o2.get(0, "d")).max() > 0 and o2.ema_variance(0) == (0.0, 0.0)


# ---- P9: elementwise independence ---------------------------------------------------

def test_coordinate_slice_evolves_like_the_full_vector():
    R, N, T, a, b = 3, 5000, 10, 1237, 3391
    w0, grads = rand_setup(R, N, T)
    full = oracle.Oracle(R, [N], p=0.2, tau=2, ema_beta=0.9, **HP)
    part = oracle.Oracle(R, [b - a], p=0.2, tau=2, ema_beta=0.9, coord_base=[a],
                         lookahead_delay=[0], **HP)
    full.init_params(0, w0); part.init_params(0, w0[a:b])
    for g in grads:
        full.step([g]); part.step([g[:, a:b]])
    for name in ("w", "m", "v", "d"):
        assert (full.get(0, name)[:, a:b] == part.get(0, name)).all()
    assert part.get(0, "d").any()


# ---- odds and ends --------------------------------------------------------------------

def test_mean_params_and_step_count_and_schedules():
    R, N = 3, 100
    w0, grads = rand_setup(R, N, 3)
    o = oracle.Oracle(R, [N], p=0.5, tau=1, ema_beta=0.9, **HP)
    o.init_params(0, w0)
    o2 = oracle.Oracle(R, [N], p=0.5, tau=1, ema_beta=0.123, **dict(HP, lr=1.0))
    o2.init_params(0, w0)
    for g in grads:
        o.step([g])
        o2.step([g], ema_beta_t=0.9, lr_t=HP["lr"])   # per-step overrides
    assert o.step_count == 3
    assert (o.mean_params(0) == seq_mean_f32(o.get(0, "w"))).all()
    # wd enters as lr_t * wd, so the overridden run equals the constant one
    assert (o.get(0, "w") == o2.get(0, "w")).all()
    assert (o.get(0, "d") == o2.get(0, "d")).all()
