"""Brute-force scalar re-statement of the block, Algorithm 1 and Algorithm 2 (pure Python loops,
Python floats = fp64, no numpy arithmetic).  Used only to pin oracle/snlp_oracle.py on tiny
inputs: it is written independently, token by token and element by element, so that an index,
sign or transposition mistake in the vectorised oracle shows up as a mismatch.
Batch size 1 only.
"""
import math


def _rms(v, eps):
    s = 0.0
    for x in v:
        s += x * x
    r = 1.0 / math.sqrt(s / len(v) + eps)
    return [x * r for x in v]


def _matvec(Wm, v):
    """Wm: list of rows (out x in)."""
    out = []
    for row in Wm:
        s = 0.0
        for j in range(len(v)):
            s += float(row[j]) * v[j]
        out.append(s)
    return out


def _rope(vec, pos, base):
    hd = len(vec)
    half = hd // 2
    out = [0.0] * hd
    for i in range(half):
        th = pos * base ** (-2.0 * i / hd)
        c, s = math.cos(th), math.sin(th)
        out[i] = vec[i] * c - vec[i + half] * s
        out[i + half] = vec[i] * s + vec[i + half] * c
    return out


class NaiveModel:
    def __init__(self, cfg, W):
        self.cfg = cfg
        self.W = W

    # ---- branches on one sequence: xs = list over t of d-vectors -------------
    def attn(self, l, xs, pos0=0, cache=None):
        c = self.cfg
        d, H, hd = c.d_model, c.n_head, c.head_dim
        Wqkv = self.W.wqkv[l]
        Wo = self.W.wo[l]
        ks = [] if cache is None else cache[0]
        vs = [] if cache is None else cache[1]
        del ks[pos0:], vs[pos0:]
        qs = []
        for t, x in enumerate(xs):
            xn = _rms(x, c.rms_eps)
            qkv = _matvec(Wqkv, xn)
            q, k, v = qkv[0:d], qkv[d:2 * d], qkv[2 * d:3 * d]
            qh, kh, vh = [], [], []
            for h in range(H):
                qh.append(_rms(_rope(q[h * hd:(h + 1) * hd], pos0 + t, c.rope_base), c.rms_eps))
                kh.append(_rms(_rope(k[h * hd:(h + 1) * hd], pos0 + t, c.rope_base), c.rms_eps))
                vh.append(v[h * hd:(h + 1) * hd])
            qs.append(qh)
            ks.append(kh)
            vs.append(vh)
        outs = []
        for t in range(len(xs)):
            o = []
            for h in range(H):
                sc = []
                for s in range(pos0 + t + 1):
                    dot = 0.0
                    for e in range(hd):
                        dot += qs[t][h][e] * ks[s][h][e]
                    sc.append(dot / math.sqrt(hd))
                mx = max(sc)
                ex = [math.exp(z - mx) for z in sc]
                Z = sum(ex)
                for e in range(hd):
                    acc = 0.0
                    for s in range(pos0 + t + 1):
                        acc += ex[s] / Z * vs[s][h][e]
                    o.append(acc)
            outs.append(_matvec(Wo, o))
        return outs

    def mlp(self, l, us):
        c = self.cfg
        outs = []
        for u in us:
            y = _matvec(self.W.wup[l], _rms(u, c.rms_eps))
            z = [max(v, 0.0) ** 2 for v in y]
            outs.append(_matvec(self.W.wdn[l], z))
        return outs

    # ---- block on streams: X = list over t of n stream vectors (each d) ------
    def block(self, l, X, pos0=0, cache=None):
        c = self.cfg
        n, d = c.n_streams, c.d_model
        T = len(X)
        if n == 1:
            xs = [X[t][0] for t in range(T)]
            a = self.attn(l, xs, pos0, cache)
            us = [[xs[t][j] + a[t][j] for j in range(d)] for t in range(T)]
            m = self.mlp(l, us)
            return [[[us[t][j] + m[t][j] for j in range(d)]] for t in range(T)]
        Ra, Rm = self.W.hc_res_attn[l], self.W.hc_res_mlp[l]
        Pa, Pm = self.W.hc_pre_attn[l], self.W.hc_pre_mlp[l]
        Qa, Qm = self.W.hc_post_attn[l], self.W.hc_post_mlp[l]
        xin = [[sum(float(Pa[s]) * X[t][s][j] for s in range(n)) for j in range(d)] for t in range(T)]
        a = self.attn(l, xin, pos0, cache)
        Xp = [[[sum(float(Ra[r][s]) * X[t][s][j] for s in range(n)) + float(Qa[r]) * a[t][j]
                for j in range(d)] for r in range(n)] for t in range(T)]
        uin = [[sum(float(Pm[s]) * Xp[t][s][j] for s in range(n)) for j in range(d)] for t in range(T)]
        m = self.mlp(l, uin)
        return [[[sum(float(Rm[r][s]) * Xp[t][s][j] for s in range(n)) + float(Qm[r]) * m[t][j]
                  for j in range(d)] for r in range(n)] for t in range(T)]

    def sequential(self, X0):
        tr = [X0]
        for l in range(self.cfg.n_layer):
            tr.append(self.block(l, tr[-1]))
        return tr

    def snlp(self, X0, K, mode):
        """Algorithm 2, S = 0, h0 init; mode 0 = identity surrogate, 1 = Hres_mlp Hres_attn, 2 = zero."""
        c = self.cfg
        L, n, d = c.n_layer, c.n_streams, c.d_model
        T = len(X0)
        old = [X0 for _ in range(L + 1)]
        for _ in range(K):
            tilde = [None] + [self.block(l, old[l]) for l in range(L)]
            new = [X0]
            for l in range(L):
                if mode == 0 or (mode == 1 and n == 1):
                    A = [[1.0 if r == s else 0.0 for s in range(n)] for r in range(n)]
                elif mode == 1:
                    Ra, Rm = self.W.hc_res_attn[l], self.W.hc_res_mlp[l]
                    A = [[sum(float(Rm[r][q]) * float(Ra[q][s]) for q in range(n)) for s in range(n)]
                         for r in range(n)]
                else:
                    A = [[0.0] * n for _ in range(n)]
                nxt = []
                for t in range(T):
                    row = []
                    for r in range(n):
                        row.append([tilde[l + 1][t][r][j]
                                    + sum(A[r][s] * (new[l][t][s][j] - old[l][t][s][j]) for s in range(n))
                                    for j in range(d)])
                    nxt.append(row)
                new.append(nxt)
            old = new
        return old

    # ---- model entry and exit (Alg. 1 lines 1 and 5) ---------------------------
    def embed(self, ids):
        """ids: list of T token ids -> list[t][s][j]; the embedding row goes into every stream."""
        c = self.cfg
        out = []
        for tok in ids:
            row = [float(self.W.embed[tok][j]) for j in range(c.d_model)]
            out.append([list(row) for _ in range(c.n_streams)])
        return out

    def lm_head(self, X):
        """X: list[t][s][j] -> logits list[t][v]: streams summed, weight-free RMSNorm (eps inside the root),
        one dot product per vocabulary row."""
        c = self.cfg
        out = []
        for t in range(len(X)):
            summed = [0.0] * c.d_model
            for s in range(c.n_streams):
                for j in range(c.d_model):
                    summed[j] += X[t][s][j]
            ms = 0.0
            for j in range(c.d_model):
                ms += summed[j] * summed[j]
            r = 1.0 / math.sqrt(ms / c.d_model + c.rms_eps)
            logits = []
            for v in range(c.vocab):
                acc = 0.0
                for j in range(c.d_model):
                    acc += float(self.W.lm_head[v][j]) * (summed[j] * r)
                logits.append(acc)
            out.append(logits)
        return out
