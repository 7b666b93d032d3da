"""Definition-level restatement of the AsyncMesh update for tiny cases.

Written separately from the C oracle, straight from the paper's equations, with
an explicit record of every past local iterate and every past subset instead of
a ring: Eq. "sparta" (Section 2.3) for the local step, Eq. "asparta" (Section
3.1) for the delayed average, Eq. "ema" and the corrected averaging (Section
3.2) for the staleness estimate, Section 2.2 for the look-ahead.  Pure Python
loops over scalars; ``ft`` picks the scalar type (numpy float32 rounds after
every operation, float64 gives a high-precision trace).  Its Philox is its own
(Python integers).
"""
import numpy as np

M32 = 0xFFFFFFFF


def philox(ctr, key):
    c = list(ctr)
    k = list(key)
    for _ in range(10):
        hi0, lo0 = divmod(0xD2511F53 * c[0], 1 << 32)
        hi1, lo1 = divmod(0xCD9E8D57 * c[2], 1 << 32)
        c = [hi1 ^ c[1] ^ k[0], lo1, hi0 ^ c[3] ^ k[1], lo0]
        k = [(k[0] + 0x9E3779B9) & M32, (k[1] + 0xBB67AE85) & M32]
    return c


def in_subset(seed, p, stage, step, mu):
    x = philox([mu >> 2, stage, step & M32, 0], [seed & M32, seed >> 32])
    return x[mu & 3] < int(np.floor(p * 4294967296.0))


def to_wire(ft, x, wire):
    """A value as sent to the other replicas: unchanged, or rounded to bfloat16 / to
    8-bit floating point (E4M3) by the tensor library's own conversion."""
    if wire == "fp32":
        return x
    import torch
    low = {"bf16": torch.bfloat16, "fp8": torch.float8_e4m3fn}[wire]
    return ft(torch.tensor(float(x), dtype=torch.float32).to(low).to(torch.float32).item())


def run(ft, R, N, p, tau, lam, lr, b1, b2, eps, wd, seed, delay, w0, grads,
        stage=0, interval=1, wire="fp32", correction="ema", keeps_own_copy=True):
    """grads[t-1][i][mu] for t = 1..T.  Returns a list of per-step records.
    keeps_own_copy: a replica still has the unrounded value it sent tau steps ago for
    its staleness sample; False: only what went over the wire exists, for everybody."""
    T = len(grads)
    w = [[ft(w0[mu]) for mu in range(N)] for _ in range(R)]
    m = [[ft(0) for _ in range(N)] for _ in range(R)]
    v = [[ft(0) for _ in range(N)] for _ in range(R)]
    d = [[ft(0) for _ in range(N)] for _ in range(R)]
    hist = {}      # t -> local iterates [i][mu]
    subsets = {}   # t -> set of coordinates
    out = []
    for t in range(1, T + 1):
        ib1 = ft(1.0 / (1.0 - b1 ** float(t)))
        ib2 = ft(1.0 / (1.0 - b2 ** float(t)))
        omb1, omb2 = ft(1.0 - b1), ft(1.0 - b2)
        lrf, lrwd, epsf = ft(lr), ft(lr * wd), ft(eps)
        lamf, oml = ft(lam), ft(1.0 - lam)
        what = [[None] * N for _ in range(R)]
        wold = [[w[i][mu] for mu in range(N)] for i in range(R)]
        for i in range(R):
            for mu in range(N):
                g = ft(grads[t - 1][i][mu])
                m[i][mu] = ft(ft(b1) * m[i][mu]) + ft(omb1 * g)
                v[i][mu] = ft(ft(b2) * v[i][mu]) + ft(omb2 * ft(g * g))
                mhat = ft(m[i][mu] * ib1)
                vhat = ft(v[i][mu] * ib2)
                upd = ft(mhat / ft(ft(np.sqrt(vhat)) + epsf))
                decayed = ft(w[i][mu] - ft(lrwd * w[i][mu]))
                what[i][mu] = ft(decayed - ft(lrf * upd))
        hist[t] = what
        subsets[t] = {mu for mu in range(N) if in_subset(seed, p, stage, t, mu)}
        for mu in range(N):
            # averaging rounds are the steps K, 2K, ...; an average launched at round
            # t - tau is consumed at round t
            if t % interval == 0 and t - tau >= 1 and mu in subsets[t - tau]:
                old = hist[t - tau]
                acc = to_wire(ft, old[0][mu], wire)
                for i in range(1, R):
                    acc = ft(acc + to_wire(ft, old[i][mu], wire))
                wbar = ft(acc / ft(R))
                for i in range(R):
                    mine = old[i][mu] if keeps_own_copy else to_wire(ft, old[i][mu], wire)
                    stal = ft(what[i][mu] - mine)
                    if correction == "ema":      # Eq. "ema"
                        d[i][mu] = ft(ft(oml * d[i][mu]) + ft(lamf * stal))
                    else:                        # eager estimate, end of Section 3.2
                        d[i][mu] = ft(stal / ft(R))
                    w[i][mu] = ft(wbar + d[i][mu])
            else:
                for i in range(R):
                    w[i][mu] = what[i][mu]
        look = [[ft(w[i][mu] + ft(ft(delay) * ft(w[i][mu] - wold[i][mu])))
                 for mu in range(N)] for i in range(R)]
        out.append(dict(
            subset=sorted(subsets[t]),
            w=np.array(w, dtype=np.float64), m=np.array(m, dtype=np.float64),
            v=np.array(v, dtype=np.float64), d=np.array(d, dtype=np.float64),
            look=np.array(look, dtype=np.float64),
            what=np.array(what, dtype=np.float64)))
    return out
