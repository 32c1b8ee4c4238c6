"""Subspace construction on the GPU (Sec. 3.1.2, Eq. 1-2) against the oracle's SVD of the same sampled rows.

Singular vectors are unique only up to sign and, where singular values nearly coincide, only as a subspace; in
finite precision that makes the trailing vectors of a slowly decaying spectrum irreproducible one by one.  What is
unique is compared: the singular values, the energy the basis captures, the leading (well separated) vectors with
the sign convention; the rest is checked for validity (orthonormal columns, convergence of the eigen-residual)."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import s4r_oracle as O
from tests.helpers import to_np

pytestmark = pytest.mark.gpu


def _s4r():
    import paper_2608_00528_b200 as s4r
    return s4r


def _case(cfg_id, context, batch, tensor="k", n_iter=0):
    s4r = _s4r()
    cfg = W.scaled_config(W.get_config(cfg_id), context=context, batch=batch)
    st = W.storage_dtype(cfg)
    rank = cfg.rank_k if tensor == "k" else cfg.rank_v
    X = torch.stack([W.make_kv(cfg, 0, b, tensor) for b in range(batch)])            # [B, T, D'] storage dtype, CPU
    rows = [W.sample_rows(cfg, 0, b, tensor) for b in range(batch)]                   # absolute row indices
    idx = torch.stack([(r_ - cfg.sink_count).to(torch.int32) for r_ in rows])
    ly = s4r.Layer(batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.rank_k, cfg.rank_v, cfg.sink_count,
                   s4r.S4R_BF16 if cfg.dtype == "bf16" else s4r.S4R_F32, context)
    sigma = torch.zeros(batch, rank, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    basis = s4r.build_basis(ly, X.cuda(), idx.cuda(), rank, n_iter=n_iter, sigma=sigma, dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert basis.dtype == st and tuple(basis.shape) == (batch, cfg.d_kv, rank)
    out = []
    for b in range(batch):
        S = to_np(X[b][rows[b]])
        B_ref, sv = O.build_basis(S, rank)                                            # fp64 SVD, sign-fixed
        Sn = O.normalize_rows(S)
        out.append(dict(B=to_np(basis[b]), sig=sigma[b].double().cpu().numpy(), B_ref=B_ref, sv=sv, Sn=Sn))
    return cfg, rank, out


def _check(cfg, rank, res, sigma_tol, energy_tol, lead, lead_tol):
    ortho_tol = 6e-3 if cfg.dtype == "bf16" else 5e-5          # bf16 storage: 2^-9 per entry on 1/sqrt(D') entries
    worst = dict(sigma=0.0, ortho=0.0, energy=0.0, lead=0.0)
    for r_ in res:
        B, B_ref, sv, Sn = r_["B"], r_["B_ref"], r_["sv"], r_["Sn"]
        # singular values (unique)
        e_sig = np.abs(r_["sig"] - sv[:rank]).max() / sv[0]
        worst["sigma"] = max(worst["sigma"], e_sig)
        assert e_sig <= sigma_tol, f"singular values off by {e_sig:.2e} of sigma_1"
        # orthonormal columns (validity)
        e_or = np.abs(B.T @ B - np.eye(rank)).max()
        worst["ortho"] = max(worst["ortho"], e_or)
        assert e_or <= ortho_tol, f"columns not orthonormal: {e_or:.2e}"
        # captured energy (unique: sum of the r largest sigma^2); the rounded oracle basis is the yardstick
        e_ref = np.linalg.norm(Sn @ O.round_to_storage(B_ref, cfg.dtype)) ** 2
        e_gpu = np.linalg.norm(Sn @ B) ** 2
        worst["energy"] = max(worst["energy"], (e_ref - e_gpu) / e_ref)
        assert e_gpu >= (1.0 - energy_tol) * e_ref, f"captured energy {e_gpu:.6f} < oracle's {e_ref:.6f}"
        # sign convention on every column (after rounding to storage a negative entry may tie the largest one)
        assert np.all(B.max(axis=0) >= -B.min(axis=0))
        # leading vectors: separated by more than the arithmetic can blur, so they agree one by one
        cos = np.sum(B[:, :lead] * B_ref[:, :lead], axis=0) / np.linalg.norm(B[:, :lead], axis=0)
        worst["lead"] = max(worst["lead"], (1.0 - cos).max())
        assert np.all(cos >= 1.0 - lead_tol), f"leading vectors differ: min cos {cos.min():.6f}"
        # the whole subspace against the oracle's leading half: every oracle vector i < r/2 lies in the GPU span
        half = rank // 2
        Qg, _ = np.linalg.qr(B)
        resid = np.linalg.norm(B_ref[:, :half] - Qg @ (Qg.T @ B_ref[:, :half]), axis=0)
        assert resid.max() <= 2e-2, f"oracle vector outside the span: {resid.max():.2e}"
    return worst


def test_basis_llama_shape_keys_and_values():
    for tensor in ("k", "v"):
        cfg, rank, res = _case(1, context=8192, batch=2, tensor=tensor)
        w = _check(cfg, rank, res, sigma_tol=2e-4, energy_tol=2e-4, lead=16, lead_tol=2e-3)
        print(f"llama {tensor}: r={rank}", {k: f"{v:.2e}" for k, v in w.items()})


def test_basis_qwen_shape():
    cfg, rank, res = _case(3, context=8192, batch=2)
    w = _check(cfg, rank, res, sigma_tol=2e-4, energy_tol=2e-4, lead=16, lead_tol=2e-3)
    print(f"qwen: r={rank}", {k: f"{v:.2e}" for k, v in w.items()})


def test_basis_fp32_storage():
    cfg, rank, res = _case(0, context=4096, batch=1)
    w = _check(cfg, rank, res, sigma_tol=2e-4, energy_tol=2e-4, lead=8, lead_tol=2e-3)
    print(f"cfg0 fp32: r={rank}", {k: f"{v:.2e}" for k, v in w.items()})


def test_more_iterations_do_not_change_the_converged_part():
    _, rank, a = _case(1, context=8192, batch=1, n_iter=24)
    _, _, b = _case(1, context=8192, batch=1, n_iter=48)
    assert np.abs(a[0]["sig"] - b[0]["sig"]).max() <= 1e-4 * a[0]["sv"][0]


def test_prefill_chain_with_gpu_built_bases_reconstructs_as_well_as_the_oracles():
    """Hybrid sampling (host helper) -> s4r_build_basis -> s4r_compress, all through the library, against the oracle's
    own chain (its sampling, its SVD, its projection) on the same prompt: the low-rank reconstruction error of the
    cached rows, a quantity that does not depend on which basis of the subspace was found, must agree."""
    s4r = _s4r()
    cfg = W.scaled_config(W.get_config(1), context=6000, batch=1)
    s, r = cfg.sink_count, cfg.rank_k
    K = W.make_kv(cfg, 0, 0, "k")
    V = W.make_kv(cfg, 0, 0, "v")
    T = K.shape[0]
    ly = s4r.Layer(1, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.rank_k, cfg.rank_v, s, s4r.S4R_BF16, T)
    idx = s4r.hybrid_sample_indices(T - s, cfg.n_sampled)
    assert np.array_equal(idx.numpy(), O.hybrid_sample_indices(T - s, cfg.n_sampled))
    d_idx = idx.cuda()[None]
    d_K, d_V = K.cuda()[None], V.cuda()[None]
    BK = s4r.build_basis(ly, d_K, d_idx, cfg.rank_k)
    BV = s4r.build_basis(ly, d_V, d_idx, cfg.rank_v)
    sink_k = torch.empty(1, s, cfg.d_kv, dtype=torch.bfloat16, device="cuda")
    sink_v = torch.empty_like(sink_k)
    CK = torch.zeros(1, T, cfg.rank_k, dtype=torch.bfloat16, device="cuda")
    CV = torch.zeros(1, T, cfg.rank_v, dtype=torch.bfloat16, device="cuda")
    ln = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = s4r.alloc_workspace(ly, T, cfg.window, cfg.top_k)
    s4r.compress(ly, d_K, d_V, BK, BV, sink_k, sink_v, CK, CV, ln, workspace=ws)
    torch.cuda.synchronize()
    assert ln.item() == T - s
    for X, B_gpu, C_gpu, rank in ((K, BK, CK, cfg.rank_k), (V, BV, CV, cfg.rank_v)):
        Xn = to_np(X)[s:]
        rec_gpu = to_np(C_gpu[0, :T - s]) @ to_np(B_gpu[0]).T
        err_gpu = np.linalg.norm(Xn - rec_gpu) / np.linalg.norm(Xn)
        B_ref, _ = O.build_basis(Xn[O.hybrid_sample_indices(T - s, cfg.n_sampled)], rank)
        B_ref = O.round_to_storage(B_ref, "bf16")
        C_ref = O.round_to_storage(Xn @ B_ref, "bf16")
        err_ref = np.linalg.norm(Xn - C_ref @ B_ref.T) / np.linalg.norm(Xn)
        print(f"relative reconstruction error: library chain {err_gpu:.5f}, oracle chain {err_ref:.5f}")
        assert abs(err_gpu - err_ref) <= 2e-3 * err_ref + 1e-5


def test_rank_deficient_sample_is_reported_not_fatal():
    """All sampled rows equal: the Gram matrix has rank one, the Cholesky factorisation meets pivots that are not
    positive.  The call must come back with S4R_DEV_NUMERIC in the status word (and a valid context)."""
    s4r = _s4r()
    cfg = W.scaled_config(W.get_config(0), context=1024, batch=1)
    ly = s4r.Layer(1, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.rank_k, cfg.rank_v, cfg.sink_count,
                   s4r.S4R_F32, 1024)
    X = torch.ones(1, 1024, cfg.d_kv, dtype=torch.float32, device="cuda")
    idx = torch.arange(512, dtype=torch.int32, device="cuda")[None]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    basis = s4r.build_basis(ly, X, idx, cfg.rank_k, dev_status=status)
    torch.cuda.synchronize()
    assert status.item() & 4
    assert tuple(basis.shape) == (1, cfg.d_kv, cfg.rank_k)
    # the device is still usable
    assert float(torch.ones(4, device="cuda").sum()) == 4.0


def test_basis_rejects_what_it_cannot_do():
    s4r = _s4r()
    cfg = W.scaled_config(W.get_config(1), context=4096, batch=1)
    ly = s4r.Layer(1, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.rank_k, cfg.rank_v, cfg.sink_count,
                   s4r.S4R_BF16, 4096)
    X = torch.zeros(1, 4096, cfg.d_kv, dtype=torch.bfloat16, device="cuda")
    idx = torch.arange(100, dtype=torch.int32, device="cuda")[None]
    with pytest.raises(s4r.S4RError) as e:                       # rank + 32 > n_samples
        s4r.build_basis(ly, X, idx, 192)
    assert e.value.status == -2
    idx = torch.arange(1024, dtype=torch.int32, device="cuda")[None]
    with pytest.raises(s4r.S4RError) as e:                       # rank too large for the in-memory eigensolver
        s4r.build_basis(ly, X, idx, 256)
    assert e.value.status == -2
