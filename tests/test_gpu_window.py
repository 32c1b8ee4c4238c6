"""Windowed relevance estimation (Eq. 7, 9, 10): a FIFO of the W_q most recent projected queries scores the cache,
each row under its own causal limit, and the probabilities are averaged.  The oracle keeps its own window; the
library's window is seeded from the oracle's rows and afterwards maintained by the library itself."""
import numpy as np
import pytest
import torch

import workloads as W
from oracle import s4r_oracle as O
from tests.helpers import Problem, to_np, from_np, TOL, BAND

pytestmark = pytest.mark.gpu


def _s4r():
    import paper_2608_00528_b200 as s4r
    return s4r


def _queries(cfg, p, b, n):
    """n successive queries of sequence b (oldest first), as stored (bf16) tensors."""
    return [W.make_query(cfg, p.K[b], p.layer, b, step=i) for i in range(n)]


def _run_case(cfg, Wq, steps=2, theta=None, cache_rows=None):
    s4r = _s4r()
    p = Problem(cfg, device="cuda").upload()
    ly = p.layer_desc()
    B, G, r, s = cfg.batch, cfg.group, cfg.rank_k, cfg.sink_count
    th = cfg.rope_theta if theta is None else theta
    L = p.L if cache_rows is None else cache_rows        # a shorter cache: only the first rows count
    p.d_len.fill_(L)
    n_q = Wq + steps - 1
    qs = [_queries(cfg, p, b, n_q) for b in range(B)]
    cq = [[O.project_query(to_np(q), p.BK[b], cfg.n_kv_heads) for q in qs[b]] for b in range(B)]     # [G, r] each
    # library window: rows 1..W_q-1 hold the W_q - 1 queries before the first scored one; row 0 is dropped
    win = torch.full((B, Wq, G, r), 7.0, dtype=torch.float32, device="cuda")
    for b in range(B):
        for i in range(Wq - 1):
            win[b, i + 1] = torch.from_numpy(cq[b][i]).float()
    ws = s4r.alloc_workspace(ly, p.cap, cfg.window, cfg.top_k, score_window=Wq)
    out = torch.empty(B, cfg.n_q_heads, cfg.head_dim, device="cuda")
    sel = torch.empty(B, cfg.window + cfg.top_k, dtype=torch.int32, device="cuda")
    cnt = torch.empty(B, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    worst = 0.0
    for t in range(steps):
        cur = Wq - 1 + t
        d_q = torch.stack([qs[b][cur].to("cuda") for b in range(B)])
        before = win.clone()
        s4r.decode_step_windowed(ly, d_q, p.d_sink_k, p.d_sink_v, p.d_CK, p.d_CV, p.d_len, p.d_BK, p.d_BV, p.cap,
                                 cfg.window, cfg.top_k, win, out, sel, cnt, ws, score_window=Wq, rope_theta=th,
                                 pool_kernel=cfg.pool_kernel,
                                 pool_mode={"max": s4r.POOL_MAX, "avg": s4r.POOL_AVG}[cfg.pool_mode],
                                 group_mode={"mean": s4r.GROUP_MEAN, "max": s4r.GROUP_MAX}[cfg.group_mode],
                                 dev_status=status)
        torch.cuda.synchronize()
        assert status.item() == 0
        assert torch.equal(win[:, :-1], before[:, 1:])                       # Eq. 7: shifted by one row
        for b in range(B):
            window_rows = np.stack(cq[b][cur - Wq + 1:cur + 1], axis=1)      # [G, W_q, r], oldest first
            got_last = win[b, -1].double().cpu().numpy()
            assert np.abs(got_last - cq[b][cur]).max() <= 2e-5 * np.abs(cq[b][cur]).max()
            res = O.decode_step(to_np(qs[b][cur]), to_np(p.K[b][:s]), to_np(p.V[b][:s]), p.CK[b][:L], p.CV[b][:L], p.BK[b],
                                p.BV[b], cfg.window, cfg.top_k, kappa=cfg.pool_kernel, pool_mode=cfg.pool_mode,
                                group_mode=cfg.group_mode, theta=th, CQ_window=window_rows)
            n = int(cnt[b].item())
            got = sel[b, :n].cpu().numpy().astype(np.int64)
            assert n == res["W_eff"] + res["k_eff"] and np.all(sel[b, n:].cpu().numpy() == -1)
            ok, msg = O.selection_agrees(res["score"], res["idx"], got, res["W_eff"], res["k_eff"], BAND)
            assert ok, f"W_q={Wq} step {t} seq {b}: {msg}"
            if np.array_equal(np.sort(got), np.sort(np.asarray(res["idx"], dtype=np.int64))):
                ref = res["out"]
            else:
                ref = O.sparse_attention(to_np(qs[b][cur]), to_np(p.K[b][:s]), to_np(p.V[b][:s]), p.CK[b][:L], p.CV[b][:L],
                                         p.BK[b], p.BV[b], np.sort(got), th)
            err = O.output_error(to_np(out[b]), ref)
            assert err <= TOL[cfg.dtype], f"W_q={Wq} step {t} seq {b}: output error {err:.3e}"
            worst = max(worst, err)
    return worst


@pytest.mark.parametrize("Wq", [2, 4, 5, 8, 32])
def test_windowed_scoring_llama_shape(Wq):
    """G = 4: 8 to 128 window rows, all scored by one pair of passes (W_q = 32 fills the 128-row operand; W_q = 5
    leaves group boundaries inside the 32-column chunks the epilogue reads)."""
    cfg = W.scaled_config(W.get_config(1), context=6000 + 4, batch=2)
    err = _run_case(cfg, Wq)
    print(f"W_q={Wq} (rows {Wq * cfg.group}): max rel err {err:.3e}")


@pytest.mark.parametrize("Wq", [3, 16, 64, 96, 128])
def test_window_lengths_that_change_the_kernel_layout(Wq):
    """W_q = 16: eight-warp epilogue with four groups per column half; 64: one group per half; 96 and 128: a group
    straddles column 64, so four warps read all columns (one group per launch pair); 3: general chunk code."""
    cfg = W.scaled_config(W.get_config(1), context=3000 + 4, batch=1)
    err = _run_case(cfg, Wq, steps=1)
    print(f"W_q={Wq}: max rel err {err:.3e}")


@pytest.mark.parametrize("over,Wq", [
    (dict(context=700 + 4, batch=16), 8),                                  # nine scan CTAs per sequence
    (dict(context=3000 + 4, batch=5, rank_k=64, rank_v=64), 6),            # one 64-column block, general chunk code
    (dict(context=3000 + 4, batch=2, rank_k=256, rank_v=128), 16),         # four blocks, five ring pieces
    (dict(context=3000 + 4, batch=2, rank_k=320, rank_v=64), 4),           # the largest supported key rank
])
def test_windowed_scoring_other_geometries(over, Wq):
    cfg = W.scaled_config(W.get_config(1), **over)
    err = _run_case(cfg, Wq, steps=1)
    print(f"{over} W_q={Wq}: max rel err {err:.3e}")


def test_windowed_scoring_without_rope_and_with_average_pooling():
    cfg = W.scaled_config(W.get_config(1), context=3000 + 4, batch=1, pool_mode="avg", group_mode="max")
    err = _run_case(cfg, 8, steps=1, theta=0.0)
    print(f"W_q=8, avg pooling, group max, no RoPE: max rel err {err:.3e}")


@pytest.mark.parametrize("Wq", [4, 32])
def test_windowed_scoring_qwen_shape_group7(Wq):
    """G = 7: 28 window rows in one pair of passes; at W_q = 32 the 224 rows take two pairs (groups 0-3, 4-6)."""
    cfg = W.scaled_config(W.get_config(3), context=5000 + 4, batch=1)
    err = _run_case(cfg, Wq, steps=1 if Wq > 8 else 2)
    print(f"qwen W_q={Wq}: max rel err {err:.3e}")


def test_window_of_one_equals_the_plain_step():
    s4r = _s4r()
    cfg = W.scaled_config(W.get_config(1), context=4000 + 4, batch=2)
    p = Problem(cfg, device="cuda").upload()
    ly = p.layer_desc()
    B = cfg.batch
    mk = lambda: (torch.empty(B, cfg.n_q_heads, cfg.head_dim, device="cuda"),
                  torch.empty(B, cfg.window + cfg.top_k, dtype=torch.int32, device="cuda"),
                  torch.empty(B, dtype=torch.int32, device="cuda"))
    out1, sel1, cnt1 = mk()
    out2, sel2, cnt2 = mk()
    ws = s4r.alloc_workspace(ly, p.cap, cfg.window, cfg.top_k, score_window=2)
    s4r.decode_step(ly, p.d_q, p.d_sink_k, p.d_sink_v, p.d_CK, p.d_CV, p.d_len, p.d_BK, p.d_BV, p.cap, cfg.window,
                    cfg.top_k, out1, sel1, cnt1, ws, rope_theta=cfg.rope_theta)
    win = torch.zeros(B, 1, cfg.group, cfg.rank_k, dtype=torch.float32, device="cuda")
    s4r.decode_step_windowed(ly, p.d_q, p.d_sink_k, p.d_sink_v, p.d_CK, p.d_CV, p.d_len, p.d_BK, p.d_BV, p.cap,
                             cfg.window, cfg.top_k, win, out2, sel2, cnt2, ws, score_window=1,
                             rope_theta=cfg.rope_theta)
    torch.cuda.synchronize()
    assert torch.equal(cnt1, cnt2)
    same = sum(len(set(sel1[b].tolist()) & set(sel2[b].tolist())) for b in range(B))
    assert same >= B * (cfg.window + cfg.top_k) - 2 * B
    assert ((out1 - out2).abs().amax() / out1.abs().amax()).item() <= 1e-3


def test_window_longer_than_the_cache():
    """Window rows whose token index would be negative see nothing and add nothing (Eq. 9's mask)."""
    cfg = W.scaled_config(W.get_config(1), context=2000 + 4, batch=1, top_k=8, window=2)
    for rows, Wq in ((0, 4), (3, 4), (1, 4), (50, 4), (20, 32), (130, 32)):
        err = _run_case(cfg, Wq, steps=1, cache_rows=rows)
        print(f"L={rows}, W_q={Wq}: max rel err {err:.3e}")
        assert err <= 1e-4            # every row is selected: what is left is the attention's own rounding


@pytest.mark.parametrize("n_init", [0, 3, 8])
def test_window_initialised_from_prompt_queries(n_init):
    """Eq. 4: the library projects the last prompt queries itself; the rows must equal the oracle's projections and
    the first windowed step on that window must agree with the oracle's step on the same rows."""
    s4r = _s4r()
    Wq = 8
    cfg = W.scaled_config(W.get_config(1), context=3000 + 4, batch=2)
    p = Problem(cfg, device="cuda").upload()
    ly = p.layer_desc()
    B, G, r, s = cfg.batch, cfg.group, cfg.rank_k, cfg.sink_count
    qs = [_queries(cfg, p, b, n_init + 1) for b in range(B)]
    cq = [[O.project_query(to_np(q), p.BK[b], cfg.n_kv_heads) for q in qs[b]] for b in range(B)]
    win = torch.full((B, Wq, G, r), 3.0, dtype=torch.float32, device="cuda")
    prompt_q = torch.stack([torch.stack(qs[b][:n_init]) for b in range(B)]).to("cuda") if n_init else None
    s4r.window_init(ly, prompt_q, p.d_BK, win, score_window=Wq)
    torch.cuda.synchronize()
    got = win.double().cpu().numpy()
    for b in range(B):
        assert np.all(got[b, :Wq - n_init] == 0.0)
        for i in range(n_init):
            ref = cq[b][i]
            assert np.abs(got[b, Wq - n_init + i] - ref).max() <= 2e-5 * np.abs(ref).max()
    ws = s4r.alloc_workspace(ly, p.cap, cfg.window, cfg.top_k, score_window=Wq)
    out = torch.empty(B, cfg.n_q_heads, cfg.head_dim, device="cuda")
    sel = torch.empty(B, cfg.window + cfg.top_k, dtype=torch.int32, device="cuda")
    cnt = torch.empty(B, dtype=torch.int32, device="cuda")
    d_q = torch.stack([qs[b][n_init].to("cuda") for b in range(B)])
    s4r.decode_step_windowed(ly, d_q, p.d_sink_k, p.d_sink_v, p.d_CK, p.d_CV, p.d_len, p.d_BK, p.d_BV, p.cap, cfg.window,
                             cfg.top_k, win, out, sel, cnt, ws, score_window=Wq, rope_theta=cfg.rope_theta)
    torch.cuda.synchronize()
    for b in range(B):
        rows = [np.zeros((G, r))] * (Wq - 1 - n_init) + cq[b][max(0, n_init - (Wq - 1)):n_init + 1]
        window_rows = np.stack(rows[-Wq:], axis=1)                               # [G, W_q, r], oldest first
        res = O.decode_step(to_np(qs[b][n_init]), to_np(p.K[b][:s]), to_np(p.V[b][:s]), p.CK[b], p.CV[b], p.BK[b], p.BV[b],
                            cfg.window, cfg.top_k, kappa=cfg.pool_kernel, pool_mode=cfg.pool_mode,
                            group_mode=cfg.group_mode, theta=cfg.rope_theta, CQ_window=window_rows)
        n = int(cnt[b].item())
        got_idx = sel[b, :n].cpu().numpy().astype(np.int64)
        ok, msg = O.selection_agrees(res["score"], res["idx"], got_idx, res["W_eff"], res["k_eff"], BAND)
        assert ok, f"seq {b}: {msg}"


@pytest.mark.parametrize("Wq", [4, 32])
def test_many_windowed_steps_stay_in_step(Wq):
    """The scoring kernels hand tiles between a producer, two issuing warps and eight epilogue warps through
    phase-parity barriers; a role that fell out of step would wait out its bound and raise S4R_DEV_TIMEOUT.  With
    the same query every step the window becomes constant after W_q steps, and so must every result bit."""
    s4r = _s4r()
    cfg = W.scaled_config(W.get_config(1), context=20000 + 4, batch=2)
    p = Problem(cfg, device="cuda").upload()
    ly = p.layer_desc()
    B = cfg.batch
    ws = s4r.alloc_workspace(ly, p.cap, cfg.window, cfg.top_k, score_window=Wq)
    win = torch.zeros(B, Wq, cfg.group, cfg.rank_k, dtype=torch.float32, device="cuda")
    out = torch.empty(B, cfg.n_q_heads, cfg.head_dim, device="cuda")
    sel = torch.empty(B, cfg.window + cfg.top_k, dtype=torch.int32, device="cuda")
    cnt = torch.empty(B, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ref = None
    for t in range(Wq + 200):
        s4r.decode_step_windowed(ly, p.d_q, p.d_sink_k, p.d_sink_v, p.d_CK, p.d_CV, p.d_len, p.d_BK, p.d_BV, p.cap,
                                 cfg.window, cfg.top_k, win, out, sel, cnt, ws, score_window=Wq,
                                 rope_theta=cfg.rope_theta, dev_status=status)
        if t == Wq:
            ref = (out.clone(), sel.clone(), cnt.clone())
        elif t > Wq and t % 20 == 0:
            assert torch.equal(out, ref[0]) and torch.equal(sel, ref[1]) and torch.equal(cnt, ref[2]), f"step {t}"
    torch.cuda.synchronize()
    assert status.item() == 0
    assert torch.equal(out, ref[0]) and torch.equal(sel, ref[1])


def test_fused_append_and_windowed_step_agrees_with_separate_calls():
    s4r = _s4r()
    Wq = 8
    cfg = W.scaled_config(W.get_config(1), context=4000 + 3, batch=2)
    res = []
    for fused in (False, True):
        p = Problem(cfg, device="cuda", capacity=cfg.cache_len + 4).upload()
        ly = p.layer_desc()
        ws = s4r.alloc_workspace(ly, p.cap, cfg.window, cfg.top_k, score_window=Wq)
        win = torch.zeros(cfg.batch, Wq, cfg.group, cfg.rank_k, dtype=torch.float32, device="cuda")
        out = torch.empty(cfg.batch, cfg.n_q_heads, cfg.head_dim, device="cuda")
        sel = torch.empty(cfg.batch, cfg.window + cfg.top_k, dtype=torch.int32, device="cuda")
        cnt = torch.empty(cfg.batch, dtype=torch.int32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        for step in (1, 2, 3):
            kt = torch.stack([W.make_token(cfg, 0, b, "k", step, "cuda") for b in range(cfg.batch)])
            vt = torch.stack([W.make_token(cfg, 0, b, "v", step, "cuda") for b in range(cfg.batch)])
            kw = dict(score_window=Wq, rope_theta=cfg.rope_theta, dev_status=status)
            if fused:
                s4r.append_decode_step_windowed(ly, kt, vt, p.d_q, p.d_sink_k, p.d_sink_v, p.d_CK, p.d_CV, p.d_len, p.d_BK,
                                                p.d_BV, p.cap, cfg.window, cfg.top_k, win, out, sel, cnt, ws, **kw)
            else:
                s4r.append(ly, kt, vt, p.d_BK, p.d_BV, p.d_CK, p.d_CV, p.d_len)
                s4r.decode_step_windowed(ly, p.d_q, p.d_sink_k, p.d_sink_v, p.d_CK, p.d_CV, p.d_len, p.d_BK, p.d_BV, p.cap,
                                         cfg.window, cfg.top_k, win, out, sel, cnt, ws, **kw)
        torch.cuda.synchronize()
        assert status.item() == 0
        res.append((out.clone(), sel.clone(), cnt.clone(), p.d_CK.clone(), p.d_len.clone(), win.clone()))
    (out_a, sel_a, cnt_a, ck_a, len_a, win_a), (out_b, sel_b, cnt_b, ck_b, len_b, win_b) = res
    assert len_a.tolist() == len_b.tolist() == [cfg.cache_len + 3] * cfg.batch
    assert torch.equal(cnt_a, cnt_b) and torch.equal(win_a, win_b)
    xf, yf = ck_a.float(), ck_b.float()
    assert torch.all((xf - yf).abs() <= 2.0 ** -7 * torch.maximum(xf.abs(), yf.abs()) + 1e-30)
    same = sum(len(set(sel_a[b].tolist()) & set(sel_b[b].tolist())) for b in range(cfg.batch))
    assert same >= cfg.batch * (cfg.window + cfg.top_k) - 2 * cfg.batch
    assert ((out_a - out_b).abs().amax() / out_a.abs().amax()).item() <= 1e-3


def test_windowed_entry_rejects_what_it_cannot_do():
    s4r = _s4r()
    cfg = W.scaled_config(W.get_config(1), context=1000 + 4, batch=1)
    p = Problem(cfg, device="cuda").upload()
    ly = p.layer_desc()
    out = torch.empty(1, cfg.n_q_heads, cfg.head_dim, device="cuda")
    sel = torch.empty(1, cfg.window + cfg.top_k, dtype=torch.int32, device="cuda")
    cnt = torch.empty(1, dtype=torch.int32, device="cuda")
    ws = s4r.alloc_workspace(ly, p.cap, cfg.window, cfg.top_k, score_window=8)
    win = torch.zeros(1, 129, cfg.group, cfg.rank_k, dtype=torch.float32, device="cuda")   # W_q > 128
    with pytest.raises(s4r.S4RError) as e:
        s4r.decode_step_windowed(ly, p.d_q, p.d_sink_k, p.d_sink_v, p.d_CK, p.d_CV, p.d_len, p.d_BK, p.d_BV, p.cap,
                                 cfg.window, cfg.top_k, win, out, sel, cnt, ws, score_window=129)
    assert e.value.status == -2
    with pytest.raises(s4r.S4RError) as e:                                                  # plain entry: W_q must be 1
        s4r.decode_step(ly, p.d_q, p.d_sink_k, p.d_sink_v, p.d_CK, p.d_CV, p.d_len, p.d_BK, p.d_BV, p.cap, cfg.window,
                        cfg.top_k, out, sel, cnt, ws, score_window=2)
    assert e.value.status == -2
