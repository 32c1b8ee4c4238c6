"""Plain fp64 CPU oracle for the S4R prefill projection and decode step.

TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement
of what the CUDA library must compute.  Nothing in the product path may import
it; it imports nothing from the product package and shares no code with it.

Every function follows one passage of the paper (arXiv 2608.00528).  Equations
in Sec. 3 of the paper are unnumbered; here "Eq. n" is the n-th displayed
equation of Sec. 3 in order of appearance:

  Eq. 1  token-wise normalisation of the sampled rows        (Sec. 3.1.2)
  Eq. 2  truncated SVD -> bases B^K, B^V                      (Sec. 3.1.2)
  Eq. 3  coefficients C = S B                                 (Sec. 3.1.2)
  Eq. 4  initial query window C^Q = Q~ B^K                    (Sec. 3.1.3)
  Eq. 5  per-step projections c_t^{Q/K} = s_t B^K, c_t^V = s_t B^V   (Sec. 3.2.1)
  Eq. 6  append to the coefficient cache                      (Sec. 3.2.1)
  Eq. 7  query-coefficient FIFO                               (Sec. 3.2.1)
  Eq. 8  latent logits Z = C^Q (C^K)^T / sqrt(r)              (Sec. 3.2.2)
  Eq. 9  causal mask + softmax over the cache length          (Sec. 3.2.2)
  Eq. 10 mean over the query window                           (Sec. 3.2.2)
  Eq. 11 sequence pooling with kernel kappa                   (Sec. 3.2.3)
  Eq. 12 group aggregation                                    (Sec. 3.2.3)
  Eq. 13 local window, Eq. 14 global top-k, Eq. 15 union      (Sec. 3.2.3)
  Eq. 16 sparse reconstruction, Eq. 17 sink concatenation     (Sec. 3.2.3)
  Eq. 18 final attention with RoPE at original positions      (Sec. 3.2.3)

All arithmetic is numpy float64.  Inputs that are stored in bf16 or fp32 are
widened exactly before they get here; results that the method *stores*
(coefficients) are rounded once, to nearest-even, into the storage type.

Readings taken where the paper is silent (listed again in the design notes):
  * projection uses the raw rows, normalisation is applied to the sampled rows only (Eq. 1 vs Eq. 3);
  * bases live in the concatenated space D' = h_kv * d_h, one per sequence and tensor (App. A);
  * Q~[g] is the concatenation over KV heads kv of query head kv*G+g, so each head meets its own KV head;
  * pooling: stride 1, same length, half-width floor(kappa/2), over the whole cache before the
    candidate slice; max ignores out-of-range neighbours, avg divides by kappa (zero padding);
    pooling per group member first, then aggregation over the group (order of Eq. 11, 12);
  * top-k ties go to the lower index; k_eff = min(k, L - W_eff), W_eff = min(W, L);
  * RoPE pairs channel i with i + d_h/2, inv_freq_i = theta^(-2i/d_h); sink j sits at position j,
    non-sink row l at s + l, the query at s + L - 1;
  * latent logits are scaled by 1/sqrt(r), final logits by 1/sqrt(d_h);
  * the cache length L includes the current token (append first, then score);
  * local-window rows are reconstructed like any other selected row; one index set per sequence.
"""
from __future__ import annotations

import numpy as np

# --------------------------------------------------------------------------- storage rounding


def round_to_storage(x, dtype: str):
    """Round fp64 values once, to nearest-even, into 'f32' or 'bf16'; returned widened to fp64."""
    x = np.asarray(x, dtype=np.float64)
    if dtype == "f64":
        return x.copy()
    if dtype == "f32":
        return x.astype(np.float32).astype(np.float64)
    if dtype == "bf16":
        # bf16 keeps 8 significant bits: x = m * 2^e with m in [0.5, 1)  ->  rint(m * 2^8) * 2^(e-8)
        m, e = np.frexp(x)
        return np.ldexp(np.rint(m * 256.0), e - 8)
    raise ValueError(dtype)


def storage_ulp(x, dtype: str):
    """Spacing of the storage grid at |x| (fp64 array)."""
    x = np.abs(np.asarray(x, dtype=np.float64))
    bits = {"f32": 24, "bf16": 8}[dtype]
    _, e = np.frexp(np.maximum(x, np.finfo(np.float64).tiny))
    return np.ldexp(1.0, e - bits)


# --------------------------------------------------------------------------- setup (Sec. 3.1)


def hybrid_sample_indices(n_nonsink: int, n_samples: int, recent_frac: float = 0.7):
    """Sec. 3.1.2 sampling in the paper's own mode: an evenly spread set over the early non-sink positions
    plus a contiguous block of the most recent ones (7:3 recent-to-uniform split in the experiments).
    Returns sorted non-sink indices in [0, n_nonsink)."""
    n_samples = min(n_samples, n_nonsink)
    n_recent = min(n_samples, int(np.ceil(recent_frac * n_samples)))
    n_uniform = n_samples - n_recent
    early_len = n_nonsink - n_recent
    recent = np.arange(early_len, n_nonsink)
    if n_uniform > 0 and early_len > 0:
        early = np.unique(np.floor(np.arange(n_uniform) * (early_len / n_uniform)).astype(np.int64))
    else:
        early = np.empty(0, dtype=np.int64)
    return np.concatenate([early, recent])


def normalize_rows(S):
    """Eq. 1: each sampled row divided by its L2 norm over the feature dimension."""
    S = np.asarray(S, dtype=np.float64)
    nrm = np.sqrt(np.sum(S * S, axis=-1, keepdims=True))
    return S / np.maximum(nrm, 1e-12)


def build_basis(S_sampled, r: int):
    """Eq. 1 + Eq. 2: B [D', r] = top-r right singular vectors of the normalised sampled rows.
    Each column's sign is fixed so its largest-magnitude entry is positive (SVD leaves it free)."""
    Sn = normalize_rows(S_sampled)
    _, sv, Zt = np.linalg.svd(Sn, full_matrices=False)
    B = Zt[:r].T.copy()
    top = np.argmax(np.abs(B), axis=0)
    sgn = np.sign(B[top, np.arange(B.shape[1])])
    sgn[sgn == 0] = 1.0
    return B * sgn[None, :], sv


def compress(K, V, s: int, BK, BV, storage: str):
    """Sec. 3.1.1 + Eq. 3 for one sequence: the first s rows are kept verbatim as sinks, every other row
    is projected, C^K = S^K B^K and C^V = S^V B^V, and stored in the storage type."""
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    sink_k, sink_v = K[:s].copy(), V[:s].copy()
    CK = round_to_storage(K[s:] @ np.asarray(BK, dtype=np.float64), storage)
    CV = round_to_storage(V[s:] @ np.asarray(BV, dtype=np.float64), storage)
    return sink_k, sink_v, CK, CV


def project_token(x, B, storage: str):
    """Eq. 5 for a key or value row: c_t = s_t B, rounded into the storage type (it is appended, Eq. 6)."""
    return round_to_storage(np.asarray(x, dtype=np.float64) @ np.asarray(B, dtype=np.float64), storage)


# --------------------------------------------------------------------------- decode (Sec. 3.2)


def group_queries(q, n_kv_heads: int):
    """Q~ [G, D'] from query heads q [H_q, d_h]: Q~[g] = concat over kv of head kv*G + g."""
    q = np.asarray(q, dtype=np.float64)
    H, dh = q.shape
    G = H // n_kv_heads
    Qt = np.empty((G, n_kv_heads * dh))
    for g in range(G):
        for kv in range(n_kv_heads):
            Qt[g, kv * dh:(kv + 1) * dh] = q[kv * G + g]
    return Qt


def project_query(q, BK, n_kv_heads: int):
    """Eq. 5 for the query: c^Q [G, r] = Q~ B^K (kept in full precision; it is not stored in the cache)."""
    return group_queries(q, n_kv_heads) @ np.asarray(BK, dtype=np.float64)


def latent_logits(CQ, CK):
    """Eq. 8: Z[g, w, l] = <C^Q[g, w], C^K[l]> / sqrt(r).  CQ is [G, W_q, r], CK is [L, r]."""
    CQ = np.asarray(CQ, dtype=np.float64)
    CK = np.asarray(CK, dtype=np.float64)
    r = CK.shape[1]
    return np.einsum("gwr,lr->gwl", CQ, CK) / np.sqrt(r)


def relevance(Z):
    """Eq. 9 + Eq. 10.  Z is [G, W_q, L]; FIFO row i (oldest first) belongs to the token at non-sink index
    L - W_q + i and may only see positions l <= L - W_q + i.  Returns A^Q [G, L]."""
    G, Wq, L = Z.shape
    A = np.zeros_like(Z)
    for i in range(Wq):
        last = L - Wq + i                      # last visible index for this query row
        if last < 0:
            continue
        z = Z[:, i, :last + 1]
        e = np.exp(z - z.max(axis=-1, keepdims=True))
        A[:, i, :last + 1] = e / e.sum(axis=-1, keepdims=True)
    return A.sum(axis=1) / Wq


def pool_sequence(A, kappa: int, mode: str):
    """Eq. 11: stride-1 pooling along the sequence with kernel kappa (odd), same output length."""
    A = np.asarray(A, dtype=np.float64)
    if kappa <= 1:
        return A.copy()
    h = kappa // 2
    G, L = A.shape
    out = np.empty_like(A)
    for l in range(L):
        lo, hi = max(0, l - h), min(L, l + h + 1)
        if mode == "max":
            out[:, l] = A[:, lo:hi].max(axis=1)
        elif mode == "avg":
            out[:, l] = A[:, lo:hi].sum(axis=1) / kappa
        else:
            raise ValueError(mode)
    return out


def pool_sequence_fast(A, kappa: int, mode: str):
    """Same as pool_sequence, vectorised over l for long caches (max is identical; avg sums the same
    neighbours, so it agrees up to fp64 summation order)."""
    A = np.asarray(A, dtype=np.float64)
    if kappa <= 1:
        return A.copy()
    h = kappa // 2
    G, L = A.shape
    pad = -np.inf if mode == "max" else 0.0
    P = np.full((G, L + 2 * h), pad)
    P[:, h:h + L] = A
    if mode == "max":
        out = P[:, 0:L].copy()
        for j in range(1, kappa):
            np.maximum(out, P[:, j:j + L], out=out)
        return out
    out = P[:, 0:L].copy()
    for j in range(1, kappa):
        out += P[:, j:j + L]
    return out / kappa


def aggregate_group(At, mode: str):
    """Eq. 12: mean or max over the group dimension -> score [L]."""
    if mode == "mean":
        return At.sum(axis=0) / At.shape[0]
    if mode == "max":
        return At.max(axis=0)
    raise ValueError(mode)


def select_indices(score, W: int, k: int):
    """Eq. 13-15: local window [L-W_eff, L) united with the k_eff best candidates of score[:L-W_eff]
    (higher score first, lower index on ties).  Returns (sorted index array, W_eff, k_eff)."""
    score = np.asarray(score, dtype=np.float64)
    L = score.shape[0]
    W_eff = min(W, L)
    n_cand = L - W_eff
    k_eff = min(max(k, 0), n_cand)
    cand = score[:n_cand]
    order = np.lexsort((np.arange(n_cand), -cand))
    glob = order[:k_eff]
    local = np.arange(n_cand, L)
    return np.sort(np.concatenate([glob, local]).astype(np.int64)), W_eff, k_eff


def rope_rotate(x, pos, theta: float):
    """RoPE (rotate-half pairing) of rows x [n, d_h] at integer positions pos [n]; theta <= 0 -> identity."""
    x = np.asarray(x, dtype=np.float64)
    if theta is None or theta <= 0:
        return x.copy()
    d = x.shape[-1]
    half = d // 2
    inv_freq = np.power(float(theta), -np.arange(half, dtype=np.float64) * 2.0 / d)
    ang = np.asarray(pos, dtype=np.float64)[:, None] * inv_freq[None, :]
    c, s = np.cos(ang), np.sin(ang)
    x1, x2 = x[:, :half], x[:, half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=1)


def sparse_attention(q, sink_k, sink_v, CK, CV, BK, BV, idx, theta: float):
    """Eq. 16-18 on a given index set `idx` (non-sink indices).  q [H_q, d_h]; sinks [s, D'];
    CK, CV [L, r]; bases [D', r].  Returns O [H_q, d_h]."""
    q = np.asarray(q, dtype=np.float64)
    sink_k = np.asarray(sink_k, dtype=np.float64)
    sink_v = np.asarray(sink_v, dtype=np.float64)
    CK = np.asarray(CK, dtype=np.float64)
    CV = np.asarray(CV, dtype=np.float64)
    BK = np.asarray(BK, dtype=np.float64)
    BV = np.asarray(BV, dtype=np.float64)
    idx = np.asarray(idx, dtype=np.int64)
    H, dh = q.shape
    s = sink_k.shape[0]
    Dp = BK.shape[0]
    h_kv = Dp // dh
    G = H // h_kv
    L = CK.shape[0]
    K_hat = CK[idx] @ BK.T                                   # Eq. 16
    V_hat = CV[idx] @ BV.T
    K_star = np.concatenate([sink_k, K_hat], axis=0)         # Eq. 17
    V_star = np.concatenate([sink_v, V_hat], axis=0)
    pos = np.concatenate([np.arange(s), s + idx])
    q_pos = np.array([s + L - 1])
    O = np.empty((H, dh))
    for h in range(H):
        kv = h // G
        Kh = rope_rotate(K_star[:, kv * dh:(kv + 1) * dh], pos, theta)
        qh = rope_rotate(q[h][None, :], q_pos, theta)[0]
        logit = Kh @ qh / np.sqrt(dh)                        # Eq. 18
        p = np.exp(logit - logit.max())
        p /= p.sum()
        O[h] = p @ V_star[:, kv * dh:(kv + 1) * dh]
    return O


def decode_step(q, sink_k, sink_v, CK, CV, BK, BV, W: int, k: int, kappa: int = 7, pool_mode: str = "max",
                group_mode: str = "mean", theta: float = 0.0, CQ_window=None, fast_pool: bool = True):
    """One decode step for one sequence (Sec. 3.2) after the current token has been appended.

    q [H_q, d_h] pre-RoPE query heads; CK/CV [L, r] coefficient caches *including* the current token;
    CQ_window: optional [G, W_q, r] query-coefficient FIFO whose last row is the current query
    (default: W_q = 1, the current query alone).
    Returns dict(out [H_q, d_h], idx (sorted), W_eff, k_eff, score [L], Z [G, W_q, L], cq [G, r]).
    """
    BK = np.asarray(BK, dtype=np.float64)
    dh = np.asarray(q).shape[1]
    h_kv = BK.shape[0] // dh
    cq = project_query(q, BK, h_kv)                          # Eq. 5
    CQ = cq[:, None, :] if CQ_window is None else np.asarray(CQ_window, dtype=np.float64)
    Z = latent_logits(CQ, CK)                                # Eq. 8
    AQ = relevance(Z)                                        # Eq. 9, 10
    pooled = (pool_sequence_fast if fast_pool else pool_sequence)(AQ, kappa, pool_mode)   # Eq. 11
    score = aggregate_group(pooled, group_mode)              # Eq. 12
    idx, W_eff, k_eff = select_indices(score, W, k)          # Eq. 13-15
    out = sparse_attention(q, sink_k, sink_v, CK, CV, BK, BV, idx, theta)   # Eq. 16-18
    return dict(out=out, idx=idx, W_eff=W_eff, k_eff=k_eff, score=score, Z=Z, cq=cq)


def dense_attention(q, K, V, theta: float, q_pos: int):
    """Textbook softmax attention of H_q query heads over full keys/values [N, D'] at positions 0..N-1
    (GQA: head h uses KV head floor(h / G)).  Used only as the closed form the invariants reduce to."""
    q = np.asarray(q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    H, dh = q.shape
    h_kv = K.shape[1] // dh
    G = H // h_kv
    N = K.shape[0]
    O = np.empty((H, dh))
    for h in range(H):
        kv = h // G
        Kh = rope_rotate(K[:, kv * dh:(kv + 1) * dh], np.arange(N), theta)
        qh = rope_rotate(q[h][None, :], np.array([q_pos]), theta)[0]
        w = Kh @ qh / np.sqrt(dh)
        w = np.exp(w - w.max())
        O[h] = (w / w.sum()) @ V[:, kv * dh:(kv + 1) * dh]
    return O


# --------------------------------------------------------------------------- comparison rules


def selection_agrees(score, idx_oracle, idx_other, W_eff: int, k_eff: int, band: float = 1e-3):
    """Index-set comparison with the tie band of the benchmark definition: let tau be the k_eff-th largest
    candidate score; a candidate j is *free* if |score_j - tau| <= band * |tau|.  The other set passes iff it
    has W_eff + k_eff distinct in-range members, contains the whole local window, contains every non-free
    index the oracle selected and no non-free index the oracle rejected.  Returns (ok, message)."""
    score = np.asarray(score, dtype=np.float64)
    L = score.shape[0]
    a = np.asarray(idx_oracle, dtype=np.int64)
    b = np.asarray(idx_other, dtype=np.int64)
    if b.size != W_eff + k_eff:
        return False, f"size {b.size} != {W_eff + k_eff}"
    if np.unique(b).size != b.size:
        return False, "duplicate indices"
    if b.size and (b.min() < 0 or b.max() >= L):
        return False, "index out of range"
    n_cand = L - W_eff
    sb = set(b.tolist())
    if any(l not in sb for l in range(n_cand, L)):
        return False, "local window incomplete"
    if k_eff == 0:
        return True, "ok"
    cand = score[:n_cand]
    tau = np.sort(cand)[::-1][k_eff - 1]
    free = np.abs(cand - tau) <= band * abs(tau)
    sa = set(a.tolist())
    for j in sa.symmetric_difference(sb):
        if j < n_cand and not free[j]:
            return False, f"index {j} differs outside the tie band (score {cand[j]:.6e}, tau {tau:.6e})"
    return True, "ok"


def output_error(out, ref):
    """Max over heads of ||out - ref||_inf / ||ref||_inf (the 'max relative error' of the benchmark)."""
    out = np.asarray(out, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    num = np.abs(out - ref).max(axis=-1)
    den = np.maximum(np.abs(ref).max(axis=-1), 1e-300)
    return float((num / den).max())
