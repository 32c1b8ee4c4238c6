"""GPU parity: the CUDA library (through its C ABI) against the fp64 oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import s4r_oracle as O
from tests.helpers import Problem, run_gpu_step, check_step, to_np, from_np, TOL

pytestmark = pytest.mark.gpu


def _s4r():
    import paper_2608_00528_b200 as s4r
    return s4r


def _cfg(i, **kw):
    return W.scaled_config(W.get_config(i), **kw)


# ------------------------------------------------------------------ decode step

@pytest.mark.parametrize("theta", [None, 0.0])
def test_decode_config0_fp32(theta):
    p = Problem(_cfg(0), device="cuda").upload()
    out, sel, cnt, status = run_gpu_step(p, theta=theta)
    assert status == 0
    err = check_step(p, out, sel, cnt, theta=theta)
    print(f"cfg0 theta={theta}: max rel err {err:.3e}")


@pytest.mark.parametrize("theta", [None, 0.0])
@pytest.mark.parametrize("value_path", [0, 1])
def test_decode_llama_shape_bf16_8k(theta, value_path):
    # config 1's layer at a context that spans several scan chunks and a ragged tail, batch 2;
    # value_path 1 = values reconstructed as in Eq. 16, 0 = library's choice (absorbed on this geometry)
    p = Problem(_cfg(1, context=8192 + 333, batch=2), device="cuda").upload()
    out, sel, cnt, status = run_gpu_step(p, theta=theta, value_path=value_path)
    assert status == 0
    err = check_step(p, out, sel, cnt, theta=theta)
    print(f"llama 8k theta={theta} value_path={value_path}: max rel err {err:.3e}")


@pytest.mark.parametrize("value_path", [0, 1])
def test_decode_qwen_shape_bf16_8k_group7(value_path):
    p = Problem(_cfg(3, context=8192 + 77, batch=2, top_k=512), device="cuda").upload()
    out, sel, cnt, status = run_gpu_step(p, value_path=value_path)
    assert status == 0
    err = check_step(p, out, sel, cnt)
    print(f"qwen 8k value_path={value_path}: max rel err {err:.3e}")


def test_decode_config1_full_size():
    p = Problem(_cfg(1), gen_device="cuda", device="cuda").upload()
    out, sel, cnt, status = run_gpu_step(p)
    assert status == 0
    err = check_step(p, out, sel, cnt)
    print(f"cfg1: max rel err {err:.3e}")
    out_b, sel_b, cnt_b, _ = run_gpu_step(p, out_dtype=torch.bfloat16)
    assert torch.equal(sel_b, sel)                                           # run-to-run determinism of selection
    assert (out_b.float() - out).abs().max() <= 2.0 ** -8 * out.abs().max() * 1.01


@pytest.mark.parametrize("pool_mode,group_mode,kappa", [("avg", "mean", 7), ("max", "max", 7), ("avg", "max", 3),
                                                        ("max", "mean", 1), ("max", "mean", 31)])
def test_decode_score_switches(pool_mode, group_mode, kappa):
    p = Problem(_cfg(0, context=3000), device="cuda").upload()
    kw = dict(pool_mode=pool_mode, group_mode=group_mode, kappa=kappa)
    out, sel, cnt, status = run_gpu_step(p, **kw)
    assert status == 0
    check_step(p, out, sel, cnt, **kw)


@pytest.mark.parametrize("Wn,k", [(64, 0), (0, 100), (5000, 10), (64, 10 ** 6), (0, 0), (1, 1), (2000, 1990)])
def test_decode_degenerate_budgets(Wn, k):
    # k = 0, W = 0, W > L, k > candidates (everything selected), nothing but sinks
    p = Problem(_cfg(0, context=2500), device="cuda").upload()
    k_arg = min(k, 4000)
    out, sel, cnt, status = run_gpu_step(p, W_=Wn, k=k_arg)
    assert status == 0
    check_step(p, out, sel, cnt, W_=Wn, k=k_arg)


def test_full_budget_equals_dense_attention_over_reconstructed_cache():
    cfg = _cfg(0, context=1500)
    p = Problem(cfg, device="cuda").upload()
    out, sel, cnt, _ = run_gpu_step(p, W_=16, k=2000)
    s = cfg.sink_count
    K_all = np.concatenate([to_np(p.K[0][:s]), p.CK[0] @ p.BK[0].T])
    V_all = np.concatenate([to_np(p.V[0][:s]), p.CV[0] @ p.BV[0].T])
    want = O.dense_attention(p.q[0], K_all, V_all, cfg.rope_theta, q_pos=s + p.L - 1)
    assert O.output_error(to_np(out[0]), want) <= TOL["f32"]
    assert int(cnt[0]) == p.L and np.array_equal(np.sort(sel[0, :p.L].cpu().numpy()), np.arange(p.L))


def test_decode_without_sinks_and_ragged_lengths():
    cfg = _cfg(1, context=5000, batch=3, sink_count=0, top_k=300)
    p = Problem(cfg, device="cuda", capacity=5100).upload()
    lens = [5000, 1234, 37]
    p.d_len = torch.tensor(lens, dtype=torch.int32, device="cuda")
    out, sel, cnt, status = run_gpu_step(p)
    assert status == 0
    for b, L in enumerate(lens):
        check_step(p, out, sel, cnt, seqs=[b], L=L)


def test_empty_cache_attends_to_sinks_only():
    cfg = _cfg(0, context=600)
    p = Problem(cfg, device="cuda").upload()
    p.d_len.zero_()
    out, sel, cnt, status = run_gpu_step(p)
    assert status == 0 and int(cnt[0]) == 0 and bool((sel == -1).all())
    s = cfg.sink_count
    ref = O.sparse_attention(p.q[0], to_np(p.K[0][:s]), to_np(p.V[0][:s]), p.CK[0][:0], p.CV[0][:0], p.BK[0], p.BV[0],
                             np.empty(0, dtype=np.int64), cfg.rope_theta)
    assert O.output_error(to_np(out[0]), ref) <= TOL["f32"]


def test_length_beyond_max_len_is_flagged_and_clamped():
    s4r = _s4r()
    p = Problem(_cfg(0, context=800), device="cuda").upload()
    p.d_len.fill_(10 ** 6)
    out, sel, cnt, status = run_gpu_step(p)
    assert status & s4r.DEV_BOUNDS
    p.d_len.fill_(p.L)
    out2, sel2, cnt2, status2 = run_gpu_step(p)
    assert status2 == 0 and torch.equal(sel, sel2)          # clamped to max_len == the true length here


def test_small_rank_head_dim_64_and_asymmetric_ranks():
    cfg = _cfg(0, context=1200, head_dim=64, n_kv_heads=4, n_q_heads=8, rank_k=8, rank_v=40, top_k=100)
    p = Problem(cfg, device="cuda").upload()
    out, sel, cnt, status = run_gpu_step(p)
    assert status == 0
    check_step(p, out, sel, cnt)


@pytest.mark.parametrize("rank_k,rank_v,value_path", [(128, 192, 0), (128, 192, 1), (128, 256, 0), (64, 128, 0)])
def test_asymmetric_ranks_with_ratio_budget_on_the_tensor_core_paths(rank_k, rank_v, value_path):
    """Sec. 3.3 / App. D: r^K < r^V and a budget given as a ratio, k = max(floor(rho L) - W, 0) (Eq. 14).  With
    r_v = 256 the absorbed kernel's tensor-memory plan does not fit and the reconstructing kernel runs."""
    s4r = _s4r()
    cfg0 = _cfg(1, context=9000 + 4, rank_k=rank_k, rank_v=rank_v)
    k = s4r.top_k_from_ratio(0.2, cfg0.cache_len, cfg0.window)
    assert k == int(0.2 * cfg0.cache_len) - cfg0.window
    cfg = _cfg(1, context=9000 + 4, rank_k=rank_k, rank_v=rank_v, top_k=k)
    p = Problem(cfg, device="cuda").upload()
    out, sel, cnt, status = run_gpu_step(p, value_path=value_path)
    assert status == 0
    err = check_step(p, out, sel, cnt)
    print(f"r_k={rank_k} r_v={rank_v} rho=0.2 (k={k}) value_path={value_path}: max rel err {err:.3e}")


def test_decode_step_host_entry_point():
    s4r = _s4r()
    cfg = _cfg(0, context=2000)
    p = Problem(cfg, device="cuda").upload()
    ly = p.layer_desc()
    ws = s4r.alloc_workspace(ly, p.cap, cfg.window, cfg.top_k)
    n = cfg.window + cfg.top_k
    q_h = p.d_q.cpu().pin_memory()
    out_h = torch.empty(1, cfg.n_q_heads, cfg.head_dim).pin_memory()
    sel_h = torch.empty(1, n, dtype=torch.int32).pin_memory()
    cnt_h = torch.empty(1, dtype=torch.int32).pin_memory()
    q_d = torch.empty_like(p.d_q)
    out_d = torch.empty(1, cfg.n_q_heads, cfg.head_dim, device="cuda")
    sel_d = torch.empty(1, n, dtype=torch.int32, device="cuda")
    cnt_d = torch.empty(1, dtype=torch.int32, device="cuda")
    s4r.decode_step_host(ly, q_h, q_d, p.d_sink_k, p.d_sink_v, p.d_CK, p.d_CV, p.d_len, p.d_BK, p.d_BV, p.cap,
                         cfg.window, cfg.top_k, out_h, out_d, sel_h, sel_d, cnt_h, cnt_d, ws,
                         rope_theta=cfg.rope_theta)
    out, sel, cnt, _ = run_gpu_step(p)
    assert torch.equal(out_h, out.cpu()) and torch.equal(sel_h, sel.cpu()) and torch.equal(cnt_h, cnt.cpu())


# ------------------------------------------------------------------ compress and append

def _check_coefficients(got: torch.Tensor, want: np.ndarray, dtype: str, absdot: np.ndarray):
    """`absdot` = sum_d |x_d| |b_d| per coefficient: the library accumulates in fp32 (unit roundoff 2^-24 per
    operation, D' <= 1024 terms), the oracle in fp64, so the two pre-rounding values differ by at most about
    2^-18 * absdot; after rounding to storage they agree to that plus one storage ulp."""
    g = to_np(got)
    acc_err = 2.0 ** -18 * absdot
    if dtype == "bf16":
        bad = np.abs(g - want) > O.storage_ulp(want, "bf16") * 1.0001 + acc_err
        assert not bad.any(), f"{bad.sum()} coefficients differ by more than 1 ulp + accumulation error"
        assert (g != want).mean() < 0.02
    else:
        assert (np.abs(g - want) <= O.storage_ulp(want, "f32") + acc_err).all()


def _absdot(x: torch.Tensor, basis: np.ndarray) -> np.ndarray:
    return np.abs(to_np(x)) @ np.abs(basis)


@pytest.mark.parametrize("ci,ctx,B", [(0, 1500, 2), (1, 2000 + 13, 2), (3, 1100, 1), (1, 5 * 256 + 4 + 77, 3),
                                      (3, 300, 2), (1, 4 + 200, 1)])
def test_compress_matches_oracle(ci, ctx, B):
    s4r = _s4r()
    cfg = _cfg(ci, context=ctx, batch=B)
    p = Problem(cfg, device="cuda").upload()
    ly = p.layer_desc()
    s = cfg.sink_count
    sk = torch.zeros_like(p.d_sink_k); sv = torch.zeros_like(p.d_sink_v)
    ck = torch.zeros_like(p.d_CK); cv = torch.zeros_like(p.d_CV)
    ln = torch.zeros(B, dtype=torch.int32, device="cuda")
    ws = s4r.alloc_workspace(ly, p.cap, cfg.window, cfg.top_k)
    s4r.compress(ly, p.d_K, p.d_V, p.d_BK, p.d_BV, sk, sv, ck, cv, ln, workspace=ws)
    torch.cuda.synchronize()
    assert torch.equal(sk, p.d_K[:, :s]) and torch.equal(sv, p.d_V[:, :s])
    assert ln.tolist() == [ctx - s] * B
    for b in range(B):
        _check_coefficients(ck[b, :p.L], p.CK[b], cfg.dtype, _absdot(p.K[b][s:], p.BK[b]))
        _check_coefficients(cv[b, :p.L], p.CV[b], cfg.dtype, _absdot(p.V[b][s:], p.BV[b]))


def test_compress_full_rank_reconstructs_the_input():
    s4r = _s4r()
    cfg = _cfg(0, context=700, n_sampled=600)
    p = Problem(cfg, device="cuda", full_rank=True).upload()
    ly = p.layer_desc()
    ck = torch.zeros_like(p.d_CK); cv = torch.zeros_like(p.d_CV)
    ln = torch.zeros(1, dtype=torch.int32, device="cuda")
    s4r.compress(ly, p.d_K, p.d_V, p.d_BK, p.d_BV, torch.zeros_like(p.d_sink_k), torch.zeros_like(p.d_sink_v), ck, cv, ln)
    rec = to_np(ck[0]) @ p.BK[0].T
    ref = to_np(p.K[0][cfg.sink_count:])
    assert np.abs(rec - ref).max() <= 1e-4 * np.abs(ref).max()


def test_append_matches_oracle_and_respects_capacity():
    s4r = _s4r()
    cfg = _cfg(1, context=900, batch=2)
    p = Problem(cfg, device="cuda", capacity=cfg.cache_len + 2).upload()
    ly = p.layer_desc()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for step in range(3):
        kt = torch.stack([W.make_token(cfg, 0, b, "k", step + 1, "cuda") for b in range(2)])
        vt = torch.stack([W.make_token(cfg, 0, b, "v", step + 1, "cuda") for b in range(2)])
        s4r.append(ly, kt, vt, p.d_BK, p.d_BV, p.d_CK, p.d_CV, p.d_len, dev_status=status)
        torch.cuda.synchronize()
        if step < 2:
            assert status.item() == 0 and p.d_len.tolist() == [p.L + step + 1] * 2
            for b in range(2):
                want = O.project_token(to_np(kt[b]), p.BK[b], "bf16")
                _check_coefficients(p.d_CK[b, p.L + step][None], want[None], "bf16", _absdot(kt[b][None], p.BK[b]))
                want = O.project_token(to_np(vt[b]), p.BV[b], "bf16")
                _check_coefficients(p.d_CV[b, p.L + step][None], want[None], "bf16", _absdot(vt[b][None], p.BV[b]))
        else:
            assert status.item() & s4r.DEV_BOUNDS and p.d_len.tolist() == [p.L + 2] * 2


def test_multi_layer_multi_step_generation_with_append():
    """Config 4's flow at reduced size: per layer compress once, then per step append the new token and decode.
    The oracle keeps its own caches; after each append the library's new row is checked against the oracle's
    and replaced by it, so every decode comparison runs on identical inputs."""
    s4r = _s4r()
    cfg = _cfg(4, context=3000 + 17, batch=2, n_layers=2, decode_steps=5, top_k=256)
    steps = cfg.decode_steps
    for layer in range(cfg.n_layers):
        p = Problem(cfg, layer=layer, device="cuda", capacity=cfg.cache_len + steps).upload()
        ly = p.layer_desc()
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        for step in range(1, steps + 1):
            kt = torch.stack([W.make_token(cfg, layer, b, "k", step, "cuda") for b in range(cfg.batch)])
            vt = torch.stack([W.make_token(cfg, layer, b, "v", step, "cuda") for b in range(cfg.batch)])
            s4r.append(ly, kt, vt, p.d_BK, p.d_BV, p.d_CK, p.d_CV, p.d_len, dev_status=status)
            torch.cuda.synchronize()
            L = p.L + step
            assert status.item() == 0 and p.d_len.tolist() == [L] * cfg.batch
            for b in range(cfg.batch):
                ck = O.project_token(to_np(kt[b]), p.BK[b], "bf16")
                cv = O.project_token(to_np(vt[b]), p.BV[b], "bf16")
                _check_coefficients(p.d_CK[b, L - 1][None], ck[None], "bf16", _absdot(kt[b][None], p.BK[b]))
                _check_coefficients(p.d_CV[b, L - 1][None], cv[None], "bf16", _absdot(vt[b][None], p.BV[b]))
                p.CK[b] = np.concatenate([p.CK[b], ck[None]])
                p.CV[b] = np.concatenate([p.CV[b], cv[None]])
                p.d_CK[b, L - 1] = from_np(ck, p.st, "cuda")
                p.d_CV[b, L - 1] = from_np(cv, p.st, "cuda")
                q = W.make_query(cfg, p.K[b], layer, b, step=step)
                p.q[b] = to_np(q)
                p.d_q[b] = q.cuda()
            out, sel, cnt, st = run_gpu_step(p)
            assert st == 0
            check_step(p, out, sel, cnt, L=L)


def test_fused_append_decode_agrees_with_separate_calls():
    s4r = _s4r()
    cfg = _cfg(1, context=5000 + 3, batch=2)
    res = []
    for fused in (False, True):
        p = Problem(cfg, device="cuda", capacity=cfg.cache_len + 4).upload()
        ly = p.layer_desc()
        ws = s4r.alloc_workspace(ly, p.cap, cfg.window, cfg.top_k)
        out = torch.empty(cfg.batch, cfg.n_q_heads, cfg.head_dim, device="cuda")
        sel = torch.empty(cfg.batch, cfg.window + cfg.top_k, dtype=torch.int32, device="cuda")
        cnt = torch.empty(cfg.batch, dtype=torch.int32, device="cuda")
        for step in (1, 2):
            kt = torch.stack([W.make_token(cfg, 0, b, "k", step, "cuda") for b in range(cfg.batch)])
            vt = torch.stack([W.make_token(cfg, 0, b, "v", step, "cuda") for b in range(cfg.batch)])
            if fused:
                s4r.append_decode_step(ly, kt, vt, p.d_q, p.d_sink_k, p.d_sink_v, p.d_CK, p.d_CV, p.d_len, p.d_BK,
                                       p.d_BV, p.cap, cfg.window, cfg.top_k, out, sel, cnt, ws,
                                       rope_theta=cfg.rope_theta)
            else:
                s4r.append(ly, kt, vt, p.d_BK, p.d_BV, p.d_CK, p.d_CV, p.d_len)
                s4r.decode_step(ly, p.d_q, p.d_sink_k, p.d_sink_v, p.d_CK, p.d_CV, p.d_len, p.d_BK, p.d_BV, p.cap,
                                cfg.window, cfg.top_k, out, sel, cnt, ws, rope_theta=cfg.rope_theta)
        torch.cuda.synchronize()
        res.append((out.clone(), sel.clone(), cnt.clone(), p.d_CK.clone(), p.d_CV.clone(), p.d_len.clone()))
    # The two routes add the D' products of the new rows in different (each fixed) orders, so a coefficient may
    # differ by one rounding of the storage type; everything downstream agrees to the accuracy of that rounding.
    (out_a, sel_a, cnt_a, ck_a, cv_a, len_a), (out_b, sel_b, cnt_b, ck_b, cv_b, len_b) = res
    assert len_a.tolist() == len_b.tolist() == [cfg.cache_len + 2] * cfg.batch
    assert torch.equal(cnt_a, cnt_b)
    for x, y in ((ck_a, ck_b), (cv_a, cv_b)):
        xf, yf = x.float(), y.float()
        assert torch.all((xf - yf).abs() <= 2.0 ** -7 * torch.maximum(xf.abs(), yf.abs()) + 1e-30)
        assert torch.equal(x[:, :cfg.cache_len], y[:, :cfg.cache_len])           # the prompt rows are untouched
    same = sum(len(set(sel_a[b].tolist()) & set(sel_b[b].tolist())) for b in range(cfg.batch))
    assert same >= cfg.batch * (cfg.window + cfg.top_k) - 2 * cfg.batch           # at most a tie-band swap per sequence
    err = (out_a - out_b).abs().amax() / out_a.abs().amax()
    assert err <= 1e-3


def test_fused_step_with_packed_host_blocks():
    """s4r_append_decode_step_host: one copy in, the fused step, one copy out; the results in the pinned host
    block must equal those of the device-pointer call on an identical cache."""
    s4r = _s4r()
    cfg = _cfg(1, context=3000 + 3, batch=2)
    res = []
    for host in (False, True):
        p = Problem(cfg, device="cuda", capacity=cfg.cache_len + 4).upload()
        ly = p.layer_desc()
        ws = s4r.alloc_workspace(ly, p.cap, cfg.window, cfg.top_k)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        out = torch.empty(cfg.batch, cfg.n_q_heads, cfg.head_dim, device="cuda")
        sel = torch.empty(cfg.batch, cfg.window + cfg.top_k, dtype=torch.int32, device="cuda")
        cnt = torch.empty(cfg.batch, dtype=torch.int32, device="cuda")
        hs = s4r.HostStep(ly, cfg.window, cfg.top_k)
        assert hs.h2d_bytes == hs.in_host.numel() and hs.d2h_bytes == hs.out_host.numel()
        for step in (1, 2):
            kt = torch.stack([W.make_token(cfg, 0, b, "k", step, "cpu") for b in range(cfg.batch)])
            vt = torch.stack([W.make_token(cfg, 0, b, "v", step, "cpu") for b in range(cfg.batch)])
            if host:
                hs.q.copy_(p.d_q.cpu()); hs.k_t.copy_(kt); hs.v_t.copy_(vt)
                hs.out_host.fill_(0x55)
                s4r.append_decode_step_host(hs, p.d_sink_k, p.d_sink_v, p.d_CK, p.d_CV, p.d_len, p.d_BK, p.d_BV, p.cap,
                                            ws, rope_theta=cfg.rope_theta, dev_status=status)
                out, sel, cnt = hs.out.clone(), hs.sel_idx.clone(), hs.sel_count.clone()   # valid on return, no sync
            else:
                s4r.append_decode_step(ly, kt.cuda(), vt.cuda(), p.d_q, p.d_sink_k, p.d_sink_v, p.d_CK, p.d_CV, p.d_len,
                                       p.d_BK, p.d_BV, p.cap, cfg.window, cfg.top_k, out, sel, cnt, ws,
                                       rope_theta=cfg.rope_theta, dev_status=status)
                torch.cuda.synchronize()
        assert status.item() == 0
        res.append((out.cpu(), sel.cpu(), cnt.cpu(), p.d_CK.cpu(), p.d_len.cpu()))
    for x, y in zip(res[0], res[1]):
        assert torch.equal(x, y)


def test_decode_step_replayed_from_a_cuda_graph():
    """A captured step must give the same result on every replay (the per-call token of the fused projection
    cannot be used there, so the library falls back to the separate projection kernel while capturing)."""
    s4r = _s4r()
    cfg = _cfg(1, context=6000 + 4, batch=2)
    p = Problem(cfg, device="cuda").upload()
    ly = p.layer_desc()
    ws = s4r.alloc_workspace(ly, p.cap, cfg.window, cfg.top_k)
    out = torch.empty(cfg.batch, cfg.n_q_heads, cfg.head_dim, device="cuda")
    sel = torch.empty(cfg.batch, cfg.window + cfg.top_k, dtype=torch.int32, device="cuda")
    cnt = torch.empty(cfg.batch, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def step():
        s4r.decode_step(ly, p.d_q, p.d_sink_k, p.d_sink_v, p.d_CK, p.d_CV, p.d_len, p.d_BK, p.d_BV, p.cap, cfg.window,
                        cfg.top_k, out, sel, cnt, ws, rope_theta=cfg.rope_theta, dev_status=status)

    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        step()                       # warm-up outside capture (function attributes, driver entry points)
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.synchronize()
    ref = None
    for q_scale in (1.0, 0.5, 1.0):
        p.d_q.copy_(torch.stack([from_np(q * q_scale, p.st, p.device) for q in p.q]))
        out.zero_(); sel.fill_(-7); cnt.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert status.item() == 0
        if q_scale == 1.0:
            check_step(p, out, sel, cnt)
            if ref is None:
                ref = (out.clone(), sel.clone())
            else:
                assert torch.equal(out, ref[0]) and torch.equal(sel, ref[1])


@pytest.mark.parametrize("rows", [1, 50, 300])
def test_captured_step_on_a_cache_shorter_than_the_grid(rows):
    """With fewer 128-row tiles than scan CTAs some CTAs have nothing to scan; on the path with the separate
    projection kernel (taken under capture) they must still prepare their share of the query operand."""
    s4r = _s4r()
    cfg = _cfg(1, context=2000 + 4, batch=2)
    p = Problem(cfg, device="cuda").upload()
    p.d_len.fill_(rows)
    ly = p.layer_desc()
    ws = s4r.alloc_workspace(ly, p.cap, cfg.window, cfg.top_k)
    ws.fill_(0x7f)                                # whatever a skipped CTA leaves behind is far from a valid operand
    out = torch.empty(cfg.batch, cfg.n_q_heads, cfg.head_dim, device="cuda")
    sel = torch.empty(cfg.batch, cfg.window + cfg.top_k, dtype=torch.int32, device="cuda")
    cnt = torch.empty(cfg.batch, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            s4r.decode_step(ly, p.d_q, p.d_sink_k, p.d_sink_v, p.d_CK, p.d_CV, p.d_len, p.d_BK, p.d_BV, p.cap,
                            cfg.window, cfg.top_k, out, sel, cnt, ws, rope_theta=cfg.rope_theta, dev_status=status)
    graph.replay()
    torch.cuda.synchronize()
    assert status.item() == 0
    err = check_step(p, out, sel, cnt, L=rows)
    assert err <= 1e-4, f"output error {err:.3e} on a {rows}-row cache"


@pytest.mark.parametrize("theta", [None, 0.0])
def test_many_back_to_back_steps_stay_in_step(theta):
    """The kernels hand work between warp roles through phase-parity barriers; a role that fell two phases behind
    would wait out its bound and raise S4R_DEV_TIMEOUT.  Several hundred steps back to back (with and without
    the RoPE work, which changes the relative speed of the roles) must leave the status word clear and give the
    same bits every time."""
    s4r = _s4r()
    cfg = _cfg(2, context=16384 + 4, batch=8)
    p = Problem(_cfg(2, context=16384 + 4, batch=1), device="cuda").upload()      # one checked sequence ...
    B = cfg.batch
    rep = lambda t: t.expand(B, *t.shape[1:]).contiguous()                         # ... replicated over the batch
    ly = s4r.Layer(B, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.rank_k, cfg.rank_v, cfg.sink_count, s4r.S4R_BF16,
                   p.cap)
    d = dict(q=rep(p.d_q), sk=rep(p.d_sink_k), sv=rep(p.d_sink_v), ck=rep(p.d_CK), cv=rep(p.d_CV), ln=rep(p.d_len),
             bk=rep(p.d_BK), bv=rep(p.d_BV))
    ws = s4r.alloc_workspace(ly, p.cap, cfg.window, cfg.top_k)
    out = torch.empty(B, cfg.n_q_heads, cfg.head_dim, device="cuda")
    sel = torch.empty(B, cfg.window + cfg.top_k, dtype=torch.int32, device="cuda")
    cnt = torch.empty(B, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    th = cfg.rope_theta if theta is None else theta
    first = None
    for i in range(300):
        s4r.decode_step(ly, d["q"], d["sk"], d["sv"], d["ck"], d["cv"], d["ln"], d["bk"], d["bv"], p.cap, cfg.window,
                        cfg.top_k, out, sel, cnt, ws, rope_theta=th, dev_status=status)
        if i in (0, 149, 299):
            torch.cuda.synchronize()
            assert status.item() == 0
            if first is None:
                first = (out.clone(), sel.clone())
                check_step(p, out[:1], sel[:1], cnt[:1], theta=theta)
                assert all(torch.equal(out[b], out[0]) and torch.equal(sel[b], sel[0]) for b in range(1, B))
            else:
                assert torch.equal(out, first[0]) and torch.equal(sel, first[1])
