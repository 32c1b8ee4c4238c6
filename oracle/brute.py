"""Pure-Python-loop restatement of one S4R decode step, for tiny shapes only.

TEST INFRASTRUCTURE ONLY.  Written independently of `s4r_oracle.py` (scalar
loops over Python floats, `math` only, no numpy contraction) so that an index,
sign or transposition mistake in the vectorised oracle shows up as a mismatch.
It follows the same passages: per-step projection (Eq. 5), latent logits
(Eq. 8), softmax (Eq. 9, query window of one), pooling (Eq. 11), group
aggregation (Eq. 12), local window + top-k + union (Eq. 13-15), sparse
reconstruction (Eq. 16), sink concatenation (Eq. 17), RoPE and attention
(Eq. 18), with Eq. n = n-th displayed equation of Sec. 3.
"""
import math


def compress_rows(X, s, B):
    """Eq. 3 without storage rounding: rows s.. of X [T][D'] times B [D'][r]."""
    T, D, r = len(X), len(B), len(B[0])
    C = []
    for t in range(s, T):
        row = []
        for j in range(r):
            acc = 0.0
            for d in range(D):
                acc += X[t][d] * B[d][j]
            row.append(acc)
        C.append(row)
    return C


def decode_step(q, sink_k, sink_v, CK, CV, BK, BV, W, k, kappa, pool_mode, group_mode, theta):
    H, dh = len(q), len(q[0])
    D, r = len(BK), len(BK[0])
    rv = len(BV[0])
    h_kv = D // dh
    G = H // h_kv
    L = len(CK)
    s = len(sink_k)
    # Eq. 5: query coefficients; channel d of Q~[g] belongs to head (d // dh) * G + g
    cq = [[0.0] * r for _ in range(G)]
    for g in range(G):
        for j in range(r):
            acc = 0.0
            for d in range(D):
                acc += q[(d // dh) * G + g][d % dh] * BK[d][j]
            cq[g][j] = acc
    # Eq. 8-9: logits and softmax over the cache
    A = []
    for g in range(G):
        z = []
        for l in range(L):
            acc = 0.0
            for j in range(r):
                acc += cq[g][j] * CK[l][j]
            z.append(acc / math.sqrt(r))
        zmax = max(z)
        e = [math.exp(v - zmax) for v in z]
        tot = sum(e)
        A.append([v / tot for v in e])
    # Eq. 11: pooling per group member
    half = kappa // 2
    P = []
    for g in range(G):
        row = []
        for l in range(L):
            nb = [A[g][j] for j in range(l - half, l + half + 1) if 0 <= j < L]
            row.append(max(nb) if pool_mode == "max" else sum(nb) / kappa)
        P.append(row)
    # Eq. 12: aggregation over the group
    score = []
    for l in range(L):
        col = [P[g][l] for g in range(G)]
        score.append(sum(col) / G if group_mode == "mean" else max(col))
    # Eq. 13-15
    W_eff = min(W, L)
    n_cand = L - W_eff
    k_eff = min(k, n_cand)
    ranked = sorted(range(n_cand), key=lambda l: (-score[l], l))
    idx = sorted(ranked[:k_eff] + list(range(n_cand, L)))
    # Eq. 16-17
    rows_k = [list(sink_k[j]) for j in range(s)]
    rows_v = [list(sink_v[j]) for j in range(s)]
    pos = list(range(s))
    for l in idx:
        rows_k.append([sum(CK[l][j] * BK[d][j] for j in range(r)) for d in range(D)])
        rows_v.append([sum(CV[l][j] * BV[d][j] for j in range(rv)) for d in range(D)])
        pos.append(s + l)

    def rot(vec, p):
        if theta <= 0:
            return list(vec)
        hh = dh // 2
        out = [0.0] * dh
        for i in range(hh):
            ang = p * theta ** (-2.0 * i / dh)
            c, sn = math.cos(ang), math.sin(ang)
            out[i] = vec[i] * c - vec[i + hh] * sn
            out[i + hh] = vec[i + hh] * c + vec[i] * sn
        return out

    # Eq. 18
    out = []
    for h in range(H):
        kv = h // G
        qh = rot(q[h], s + L - 1)
        logits = []
        for n in range(len(rows_k)):
            kh = rot(rows_k[n][kv * dh:(kv + 1) * dh], pos[n])
            logits.append(sum(qh[i] * kh[i] for i in range(dh)) / math.sqrt(dh))
        m = max(logits)
        e = [math.exp(v - m) for v in logits]
        tot = sum(e)
        o = [0.0] * dh
        for n in range(len(rows_k)):
            w = e[n] / tot
            for i in range(dh):
                o[i] += w * rows_v[n][kv * dh + i]
        out.append(o)
    return out, idx, score
