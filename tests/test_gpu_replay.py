"""GPU replays of the cached denoising loop (Algorithm 1 / Appendix A) against the fp64 oracle:
refresh -> attend -> gate, step after step, on the same seeded tensors.  Compared per step: the
attention output (bf16: max-abs <= 1e-2; fp32: <= 1e-5 relative), the gate's maximum entropy
(<= 1e-4 nats) and decision (bit-exact unless |E - tau| < 1e-4, where the oracle's decision drives
both replays); at the end: the KV caches byte for byte."""
import numpy as np
import pytest
import torch

import ec_synth as syn
import oracle
from _replay import run_replay, run_replay_sliding, step_inputs, ReplayState, decoded_this_step
from _util import to_dev, to_f64, to_storage

pytestmark = pytest.mark.gpu


def _caches(w):
    t = syn.attn_inputs(w, w.ctx_len)
    return t["k_cache"], t["v_cache"]


def _oracle_fns(w, kc, vc):
    def attend(q, kn, vn, idx):
        return oracle.refresh_and_attend(q, kn, vn, kc, vc, idx, w.dtype)

    def gate(logits, flags, tau):
        o = oracle.entropy_gate(logits, w.dtype, w.vocab, flags, tau, w.block)
        return o["max_entropy"][0], int(o["decision"][0])

    return attend, gate


def _gpu_fns(w, gk, gv):
    import paper_2603_18489_b200 as ec

    d = ec.make_desc(w.batch, w.ctx_len, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def attend(q, kn, vn, idx):
        out = ec.ec_attend(d, to_dev(q), to_dev(kn), to_dev(vn), gk, gv, to_dev(idx), dev_status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        return to_f64(out)

    def gate(logits, flags, tau):
        r = ec.ec_entropy_gate(to_dev(logits), w.vocab, w.block, to_dev(flags), tau)
        torch.cuda.synchronize()
        return float(r["max_entropy"][0]), int(r["decision"][0])

    return attend, gate


def _compare(w, n_steps, tau, k, sigma_centre_fn=None):
    kc, vc = _caches(w)
    okc, ovc = kc.copy(), vc.copy()
    o_att, o_gate = _oracle_fns(w, okc, ovc)
    ref = run_replay(w, n_steps, tau, k, o_att, o_gate, None, sigma_centre_fn)
    forced = [r["decision"] for r in ref]
    gk, gv = to_dev(kc), to_dev(vc)
    g_att, g_gate = _gpu_fns(w, gk, gv)
    got = run_replay(w, n_steps, tau, k, g_att, g_gate, None, sigma_centre_fn, forced_decisions=forced)
    assert ref[0]["full"] and got[0]["full"]
    for a, b in zip(ref, got):
        assert a["full"] == b["full"] and a["n_active"] == b["n_active"]
        err = np.abs(a["out"] - b["out"]).max()
        if w.dtype == syn.BF16:
            assert err <= 1e-2, (a["step"], err)
        else:
            assert err <= 1e-5 * np.abs(a["out"]).max(), (a["step"], err)
        assert abs(a["E"] - b["E"]) <= 1e-4, (a["step"], a["E"], b["E"])
        if abs(a["E"] - tau) >= 1e-4:
            assert a["decision"] == b["decision"], (a["step"], a["E"], tau)
    assert np.array_equal(to_storage(gk), okc) and np.array_equal(to_storage(gv), ovc)
    return ref


def _tau_for_recompute_share(w, n_steps, share, sigma_centre_fn=None):
    """tau such that about `share` of the steps exceed it: the per-step maximum entropies only depend on the
    seeded logits and flags, so a gate-only pre-pass of the oracle gives them."""
    st = ReplayState(w)
    E = []
    for s in range(n_steps):
        centre = None if sigma_centre_fn is None else sigma_centre_fn(s)
        lg = step_inputs(w, s, 1, centre)["logits"]
        flags = decoded_this_step(st, s, 4)
        if not flags.any():
            st.masked[:] = True
            flags = decoded_this_step(st, s, 4)
        o = oracle.entropy_gate(lg, w.dtype, w.vocab, flags, 0.0, w.block)
        E.append(o["max_entropy"][0])
        st.record(flags, 0)
    return float(np.float32(np.quantile(E, 1.0 - share)))


def test_config1_eight_step_replay_fp32():
    w = syn.C1
    tau = _tau_for_recompute_share(w, 8, 0.5)          # config 1: tau = median
    ref = _compare(w, 8, tau, w.k_recent)
    kinds = [r["full"] for r in ref]
    assert kinds[0] and any(kinds[1:]) and not all(kinds)      # both branches were exercised


@pytest.mark.parametrize("k", [2, 8])
def test_config4_block_replay_with_drifting_sigma(k):
    w = syn.C4
    centre = lambda s: syn.drifting_sigma_centre(s)
    tau = _tau_for_recompute_share(w, 32, 0.15, centre)
    ref = _compare(w, 32, tau, k, centre)
    n_full = sum(r["full"] for r in ref)
    assert 2 <= n_full <= 12
    assert all(r["n_active"] in (w.ctx_len,) or 32 <= r["n_active"] <= 32 + 32 for r in ref)


@pytest.mark.parametrize("name,k,n_steps", [("c1_tiny_fp32", 2, 10), ("c2_llada_l768", 2, 12), ("c2_llada_l768", 6, 12)])
def test_loop_state_kept_on_the_device(name, k, n_steps):
    """The whole loop of Appendix A with its state on the GPU: the gate's decision tensor and the step's decoded
    flags go straight into ec_select_recent, whose row list (padded with -1 up to a fixed capacity) goes straight
    into ec_attend; the host only reads skip_flag to pick the branch.  Every step is compared with the oracle
    (attention output of the real rows, E, decision, history, row list); at the end the caches byte for byte."""
    import paper_2603_18489_b200 as ec

    w = syn.WORKLOADS[name]
    assert w.batch == 1
    dev = torch.device("cuda")
    n_cap = w.block + 8
    tau = _tau_for_recompute_share(w, n_steps, 0.3)
    kc, vc = _caches(w)
    okc, ovc = kc.copy(), vc.copy()
    gk, gv = to_dev(kc), to_dev(vc)
    d = ec.make_desc(1, w.ctx_len, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    hist, state = ec.new_history(1, w.ctx_len), ec.new_step_state(1, 1)
    idx_dev = torch.full((1, n_cap), -1, dtype=torch.int32, device=dev)
    w0 = w.prompt_len
    w0_dev = torch.tensor([w0], dtype=torch.int32, device=dev)
    H, t, dt, skip = np.full(w.ctx_len, -np.inf), 1, 0, False
    rows = None
    host = ReplayState(w)          # only for the seeded choice of which rows get decoded
    n_partial = 0
    for s in range(n_steps):
        st = state.cpu().numpy()[0]
        assert st[0] == t and st[1] == dt and st[2] == int(skip)
        if s == 0 or not skip:
            tin = step_inputs(w, s, w.ctx_len)
            out = ec.ec_attend(d, to_dev(tin["q"]), to_dev(tin["k_new"]), to_dev(tin["v_new"]), gk, gv, None, dev_status=status)
            want = oracle.refresh_and_attend(tin["q"], tin["k_new"], tin["v_new"], okc, ovc, None, w.dtype)
            got = to_f64(out)
        else:
            n_partial += 1
            assert st[3] == rows.size <= n_cap
            assert idx_dev.cpu().numpy()[0, :rows.size].tolist() == rows.tolist()
            tin = step_inputs(w, s, n_cap)     # the padded rows carry inputs too; their outputs are not used
            out = ec.ec_attend(d, to_dev(tin["q"]), to_dev(tin["k_new"]), to_dev(tin["v_new"]), gk, gv, idx_dev, dev_status=status)
            n = rows.size
            want = oracle.refresh_and_attend(tin["q"][:, :n], tin["k_new"][:, :n], tin["v_new"][:, :n], okc, ovc,
                                             rows[None, :].astype(np.int32), w.dtype)
            got = to_f64(out)[:, :n]
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        err = np.abs(want - got).max()
        assert err <= (1e-2 if w.dtype == syn.BF16 else 1e-5 * np.abs(want).max()), (s, err)
        flags = decoded_this_step(host, s, 4)
        if not flags.any():
            host.masked[:] = True
            flags = decoded_this_step(host, s, 4)
        host.record(flags, 0)
        o = oracle.entropy_gate(tin["logits"], w.dtype, w.vocab, flags, tau, w.block)
        flags_dev = to_dev(flags)
        g = ec.ec_entropy_gate(to_dev(tin["logits"]), w.vocab, w.block, flags_dev, tau)
        assert abs(float(g["max_entropy"][0]) - o["max_entropy"][0]) <= 1e-4
        assert abs(o["max_entropy"][0] - tau) >= 1e-4          # tau is a quantile of other steps' values or far away
        assert int(g["decision"][0]) == int(o["decision"][0])
        ec.ec_select_recent(hist, state, flags_dev, w0_dev, w.block, g["decision"], k, idx_dev)
        R, skip, dt, t = oracle.step_bookkeeping(H, t, dt, w0 + np.flatnonzero(flags), int(o["decision"][0]), k)
        rows = oracle.partial_step_rows(w0, w.block, R)
        want_h = np.where(np.isfinite(H), H, -(2 ** 31)).astype(np.int64)
        assert np.array_equal(hist.cpu().numpy()[0].astype(np.int64), want_h)
    assert n_partial >= 2
    assert np.array_equal(to_storage(gk), okc) and np.array_equal(to_storage(gv), ovc)


@pytest.mark.parametrize("name,window,k", [("c1_tiny_fp32", 8, 2), ("c2_llada_l768", 32, 4), ("c3_dream_l768", 32, 2),
                                            ("c2_llada_l768", 64, 8), ("c4_llada_l2048", 128, 2)])
def test_sliding_window_replay(name, window, k):
    """Sliding-window decoding (the paper's evaluation mode, window 32; its appendix varies the window from 8 to 128):
    the window is the first `window` still-masked positions, non-contiguous after the first decode, so the row lists
    are arbitrary ascending sets plus the recent rows; LLaDA and Dream (GQA) geometries."""
    w = syn.WORKLOADS[name]
    n_steps = 10
    kc, vc = _caches(w)
    okc, ovc = kc.copy(), vc.copy()
    o_att, _ = _oracle_fns(w, okc, ovc)

    def o_gate(logits, flags, tau):
        o = oracle.entropy_gate(logits, w.dtype, w.vocab, flags, tau, window)
        return o["max_entropy"][0], int(o["decision"][0])

    probe = run_replay_sliding(w, window, n_steps, 0.0, k, lambda *a: np.zeros(1), o_gate)
    tau = float(np.float32(np.quantile([r["E"] for r in probe], 0.7)))     # about a third of the steps recompute
    ref = run_replay_sliding(w, window, n_steps, tau, k, o_att, o_gate)
    gk, gv = to_dev(kc), to_dev(vc)
    g_att, _ = _gpu_fns(w, gk, gv)

    def g_gate(logits, flags, tau):
        import paper_2603_18489_b200 as ec

        r = ec.ec_entropy_gate(to_dev(logits), w.vocab, window, to_dev(flags), tau)
        torch.cuda.synchronize()
        return float(r["max_entropy"][0]), int(r["decision"][0])

    got = run_replay_sliding(w, window, n_steps, tau, k, g_att, g_gate, forced_decisions=[r["decision"] for r in ref])
    assert len(ref) == len(got) >= 6 and any(not r["full"] for r in ref[1:])
    for a, b in zip(ref, got):
        assert a["full"] == b["full"] and a["n_active"] == b["n_active"]
        err = np.abs(a["out"] - b["out"]).max()
        assert err <= (1e-2 if w.dtype == syn.BF16 else 1e-5 * np.abs(a["out"]).max()), (a["step"], err)
        assert abs(a["E"] - b["E"]) <= 1e-4
        if abs(a["E"] - tau) >= 1e-4:
            assert a["decision"] == b["decision"]
    assert np.array_equal(to_storage(gk), okc) and np.array_equal(to_storage(gv), ovc)


@pytest.mark.parametrize("name,window,k", [("c4_llada_l2048", 32, 2), ("c4_dream_l2048", 32, 4)])
def test_sliding_window_loop_state_kept_on_the_device(name, window, k):
    """The paper's own decoding mode at L = 2048, both model geometries, with nothing of the loop on the host:
    ec_entropy_gate_decode forms the decoded set and the decision, ec_select_recent_sliding updates history and mask
    and writes the next row list, ec_attend reads that list from device memory (padded with -1 up to a fixed
    capacity); the host reads skip_flag only.  Every step against the oracle: attention output (all real rows of a
    partial step, sampled rows of a full one), decoded set, E, decision, history, mask, row list; at the end the
    caches byte for byte."""
    import paper_2603_18489_b200 as ec

    w = syn.WORKLOADS[name]
    n_steps, n_cap = 9, window + k + 8
    dev = torch.device("cuda")
    V = w.vocab

    def step_logits(s):
        """Window rows: Gaussian with sigma <= 3 (confidence far below 0.9), a seeded few with one logit raised by
        20 to 26 (confidence 0.97 and up, entropy between 0.005 and 0.5 nats), so no confidence sits near the threshold."""
        d = syn.logits_rows(window, V, w.dtype, cfg_id=w.cfg_id, step=s, sigma_hi=3.0)
        x = syn.decode_f64(d["logits"], w.dtype)
        rng = np.random.Generator(np.random.PCG64(31 * s + w.cfg_id))
        for r in rng.choice(window, size=int(rng.integers(1, 5)), replace=False):
            x[r, int(rng.integers(0, V))] += 20.0 + 6.0 * rng.random()
        return syn.encode(x.astype(np.float32), w.dtype)

    ones = np.ones(window, np.uint8)
    logits = [step_logits(s) for s in range(n_steps)]
    E = sorted(float(oracle.entropy_gate_decode(lg, w.dtype, V, ones, 0.9, 0.0, window)["max_entropy"][0]) for lg in logits)
    gaps = [E[i] - E[i - 1] for i in range(n_steps // 2, n_steps - 1)]          # a third to a half of the steps recompute
    cut = n_steps // 2 + int(np.argmax(gaps))
    assert E[cut] - E[cut - 1] > 1e-3
    tau = float(np.float32(0.5 * (E[cut] + E[cut - 1])))

    kc, vc = _caches(w)
    okc, ovc = kc.copy(), vc.copy()
    gk, gv = to_dev(kc), to_dev(vc)
    d = ec.make_desc(1, w.ctx_len, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    hist, state = ec.new_history(1, w.ctx_len), ec.new_step_state(1, 1)
    M = np.zeros(w.ctx_len, np.uint8)
    M[w.prompt_len:] = 1
    masked_dev = to_dev(M.copy()[None, :])
    cur = oracle.sliding_window_rows(M, window)
    idx_dev = torch.full((1, n_cap), -1, dtype=torch.int32, device=dev)
    idx_dev[0, :window] = torch.from_numpy(cur.astype(np.int32)).to(dev)
    H, t, dt, skip = np.full(w.ctx_len, -np.inf), 1, 0, False
    rows = None
    n_partial = 0
    sample = sorted(np.random.Generator(np.random.PCG64(3)).choice(w.ctx_len, 10, replace=False).tolist() + [0, w.ctx_len - 1])
    for s in range(n_steps):
        st = state.cpu().numpy()[0]
        assert st[0] == t and st[1] == dt and st[2] == int(skip)
        if s == 0 or not skip:
            tin = step_inputs(w, s, w.ctx_len)
            out = ec.ec_attend(d, to_dev(tin["q"]), to_dev(tin["k_new"]), to_dev(tin["v_new"]), gk, gv, None, dev_status=status)
            want = oracle.refresh_and_attend(tin["q"], tin["k_new"], tin["v_new"], okc, ovc, None, w.dtype, row_sel=sample)
            got = to_f64(out[:, sample])
        else:
            n_partial += 1
            n = rows.size
            assert st[3] == n <= n_cap
            tin = step_inputs(w, s, n_cap)       # the padded rows carry inputs too; their outputs are not used
            out = ec.ec_attend(d, to_dev(tin["q"]), to_dev(tin["k_new"]), to_dev(tin["v_new"]), gk, gv, idx_dev, dev_status=status)
            want = oracle.refresh_and_attend(tin["q"][:, :n], tin["k_new"][:, :n], tin["v_new"][:, :n], okc, ovc,
                                             rows[None, :].astype(np.int32), w.dtype)
            got = to_f64(out)[:, :n]
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert np.abs(want - got).max() <= 1e-2, s
        o = oracle.entropy_gate_decode(logits[s], w.dtype, V, ones, 0.9, tau, window)
        assert not (np.abs(o["conf"] - np.float64(np.float32(0.9))) <= 1e-3).any()
        tok = torch.full((window,), -1, dtype=torch.int32, device=dev)
        g = ec.ec_entropy_gate_decode(to_dev(logits[s]), V, window, to_dev(ones.copy()), 0.9, tau, tok)
        assert np.array_equal(g["decoded"].cpu().numpy(), o["decoded"]), s
        assert abs(float(g["max_entropy"][0]) - o["max_entropy"][0]) <= 1e-4 and abs(o["max_entropy"][0] - tau) >= 1e-4
        assert int(g["decision"][0]) == int(o["decision"][0])
        ec.ec_select_recent_sliding(hist, state, masked_dev, g["decoded"], window, g["decision"], k, idx_dev)
        new_rows, skip, dt, t = oracle.sliding_step_bookkeeping(H, M, t, dt, cur, o["decoded"], int(o["decision"][0]), k, window)
        cur = new_rows[:min(window, int(M.sum()))]
        rows = new_rows
        assert np.array_equal(hist.cpu().numpy()[0].astype(np.int64), np.where(np.isfinite(H), H, -(2 ** 31)).astype(np.int64))
        assert np.array_equal(masked_dev.cpu().numpy()[0], M)
        g_idx = idx_dev.cpu().numpy()[0]
        assert g_idx[:rows.size].tolist() == rows.tolist() and np.all(g_idx[rows.size:] == -1)
    assert n_partial >= 3
    assert np.array_equal(to_storage(gk), okc) and np.array_equal(to_storage(gv), ovc)
