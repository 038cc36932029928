"""ec_select_recent against the oracle's Eq. 2-3 / Appendix A bookkeeping: bit-exact integer work.
Multi-step traces (the device keeps history and state between steps), ties at the threshold, budgets from 0 to
more than the decoded count, several context lengths (one, several and many positions per thread), padding and
truncation of the row list, an out-of-range window."""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu

NEVER = -(2 ** 31)


def _trace(B, L, block, k, n_steps, seed, n_cap, per_step_max=5, t0=1):
    import paper_2603_18489_b200 as ec

    rng = np.random.Generator(np.random.PCG64(seed))
    dev = torch.device("cuda")
    hist = ec.new_history(B, L)
    state = ec.new_step_state(B, t0)
    idx = torch.empty(B, n_cap, dtype=torch.int32, device=dev)
    H = [np.full(L, -np.inf) for _ in range(B)]
    t, dt = [t0] * B, [0] * B
    n_blocks = L // block
    w0 = None
    for s in range(n_steps):
        if s % 7 == 0:   # the window moves to another block every few steps
            w0 = rng.integers(0, n_blocks, size=B).astype(np.int32) * block
        flags = np.zeros((B, block), np.uint8)
        for b in range(B):
            n_dec = int(rng.integers(0, per_step_max + 1))
            flags[b, rng.choice(block, size=min(n_dec, block), replace=False)] = 1
        dec = rng.integers(0, 2, size=B).astype(np.int32)
        ec.ec_select_recent(hist, state, torch.from_numpy(flags.reshape(-1)).to(dev), torch.from_numpy(w0).to(dev),
                            block, torch.from_numpy(dec).to(dev), k, idx)
        torch.cuda.synchronize()
        g_hist, g_state, g_idx = hist.cpu().numpy(), state.cpu().numpy(), idx.cpu().numpy()
        for b in range(B):
            pos = int(w0[b]) + np.flatnonzero(flags[b])
            R, skip, dt[b], t[b] = oracle.step_bookkeeping(H[b], t[b], dt[b], pos, int(dec[b]), k)
            rows = oracle.partial_step_rows(int(w0[b]), block, R)
            want_h = np.where(np.isfinite(H[b]), H[b], NEVER).astype(np.int64)
            assert np.array_equal(g_hist[b].astype(np.int64), want_h), (s, b)
            assert g_state[b].tolist() == [t[b], dt[b], int(skip), rows.size], (s, b, g_state[b], rows.size)
            n_keep = min(rows.size, n_cap)
            assert g_idx[b, :n_keep].tolist() == rows[:n_keep].tolist(), (s, b)
            assert np.all(g_idx[b, n_keep:] == -1), (s, b)


@pytest.mark.parametrize("B,L,block,k", [(1, 768, 32, 2), (8, 4096, 32, 8), (2, 259, 7, 3), (3, 1024, 32, 64),
                                         (2, 768, 32, 0), (1, 6000, 32, 16), (2, 2048, 64, 200)])
def test_multi_step_traces_match_the_oracle(B, L, block, k):
    _trace(B, L, block, k, n_steps=40, seed=17 * L + k, n_cap=block + 256)


def test_longest_supported_context_and_one_beyond():
    """16384 positions (64 history entries per thread) is the limit; one more is refused by the host."""
    import paper_2603_18489_b200 as ec

    _trace(1, 16384, 32, 64, n_steps=12, seed=3, n_cap=32 + 128)
    dev = torch.device("cuda")
    z = torch.zeros(1, dtype=torch.int32, device=dev)
    with pytest.raises(ec.EcError):
        ec.ec_select_recent(ec.new_history(1, 16385), ec.new_step_state(1), torch.zeros(32, dtype=torch.uint8, device=dev),
                            z, 32, z, 2, torch.empty(1, 64, dtype=torch.int32, device=dev))


def test_row_list_is_cut_at_the_capacity_and_the_count_still_reports_the_need():
    _trace(2, 1024, 32, 64, n_steps=30, seed=5, n_cap=40, per_step_max=12)


def test_many_ties_at_the_threshold():
    """Whole blocks decoded in one step: the k-th largest value is shared by many positions, all of which belong to R."""
    _trace(2, 512, 32, 4, n_steps=25, seed=9, n_cap=32 + 480, per_step_max=32)


def test_window_outside_the_context_leaves_the_sequence_untouched():
    import paper_2603_18489_b200 as ec

    dev = torch.device("cuda")
    hist, state = ec.new_history(2, 128), ec.new_step_state(2, 1)
    idx = torch.full((2, 40), 77, dtype=torch.int32, device=dev)
    flags = torch.ones(2 * 32, dtype=torch.uint8, device=dev)
    w0 = torch.tensor([64, 100], dtype=torch.int32, device=dev)      # second window would end at 132 > 128
    ec.ec_select_recent(hist, state, flags, w0, 32, torch.zeros(2, dtype=torch.int32, device=dev), 2, idx)
    torch.cuda.synchronize()
    st = state.cpu().numpy()
    assert st[0].tolist() == [2, 1, 1, 32] and st[1].tolist() == [1, 0, 0, -1]
    assert (hist[1] == NEVER).all() and (idx[1] == 77).all()
    assert (hist[0, 64:96] == 1).all() and idx[0, :32].tolist() == list(range(64, 96))


def test_argument_errors_are_reported_by_the_host():
    import paper_2603_18489_b200 as ec

    dev = torch.device("cuda")
    hist, state = ec.new_history(1, 128), ec.new_step_state(1)
    flags = torch.zeros(32, dtype=torch.uint8, device=dev)
    z = torch.zeros(1, dtype=torch.int32, device=dev)
    with pytest.raises(ec.EcError):
        ec.ec_select_recent(hist, state, flags, z, 32, z, 129, torch.empty(1, 64, dtype=torch.int32, device=dev))   # k > L
    with pytest.raises(ec.EcError):
        ec.ec_select_recent(hist, state, flags, z, 32, z, 2, torch.empty(1, 16, dtype=torch.int32, device=dev))    # n_cap < block


def _sliding_trace(B, L, prompt, window, k, n_steps, seed, n_cap):
    import paper_2603_18489_b200 as ec

    rng = np.random.Generator(np.random.PCG64(seed))
    dev = torch.device("cuda")
    hist, state = ec.new_history(B, L), ec.new_step_state(B, 1)
    masked_np = np.ones((B, L), np.uint8)
    masked_np[:, :prompt] = 0
    masked = torch.from_numpy(masked_np.copy()).to(dev)
    idx = torch.full((B, n_cap), -1, dtype=torch.int32, device=dev)
    H = [np.full(L, -np.inf) for _ in range(B)]
    M = [masked_np[b].copy() for b in range(B)]
    cur = [oracle.sliding_window_rows(M[b], window) for b in range(B)]      # the current window of each sequence
    for b in range(B):                                                       # the caller seeds the first window
        idx[b, :cur[b].size] = torch.from_numpy(cur[b].astype(np.int32)).to(dev)
    t, dt = [1] * B, [0] * B
    for s in range(n_steps):
        flags = (rng.random((B, window)) < 0.2).astype(np.uint8)             # flags behind a shrunken window are ignored
        dec = rng.integers(0, 2, size=B).astype(np.int32)
        ec.ec_select_recent_sliding(hist, state, masked, torch.from_numpy(flags.reshape(-1)).to(dev), window,
                                    torch.from_numpy(dec).to(dev), k, idx)
        torch.cuda.synchronize()
        g_hist, g_state, g_idx, g_m = hist.cpu().numpy(), state.cpu().numpy(), idx.cpu().numpy(), masked.cpu().numpy()
        for b in range(B):
            new_rows, skip, dt[b], t[b] = oracle.sliding_step_bookkeeping(H[b], M[b], t[b], dt[b], cur[b], flags[b],
                                                                           int(dec[b]), k, window)
            cur[b] = new_rows[:min(window, int(M[b].sum()))]
            want_h = np.where(np.isfinite(H[b]), H[b], NEVER).astype(np.int64)
            assert np.array_equal(g_hist[b].astype(np.int64), want_h), (s, b)
            assert np.array_equal(g_m[b], M[b]), (s, b)
            assert g_state[b].tolist() == [t[b], dt[b], int(skip), new_rows.size], (s, b)
            n_keep = min(new_rows.size, n_cap)
            assert g_idx[b, :n_keep].tolist() == new_rows[:n_keep].tolist(), (s, b)
            assert np.all(g_idx[b, n_keep:] == -1)


@pytest.mark.parametrize("B,L,prompt,window,k", [(1, 768, 512, 32, 2), (4, 4096, 3072, 32, 64), (2, 300, 100, 8, 3),
                                                 (2, 1024, 0, 128, 16), (1, 6000, 5000, 32, 8)])
def test_sliding_window_traces_match_the_oracle(B, L, prompt, window, k):
    _sliding_trace(B, L, prompt, window, k, n_steps=30, seed=19 * L + k, n_cap=window + 512)


def test_sliding_window_runs_out_of_masked_positions():
    """40 positions to generate, window 16: after a few steps fewer than 16 remain and the window shrinks to what is left."""
    _sliding_trace(1, 140, 100, 16, 4, n_steps=40, seed=77, n_cap=16 + 64)


def test_sliding_window_list_that_is_not_masked_positions_is_rejected_per_sequence():
    """Sequence 0 is seeded with its proper first window, sequence 1 with a list that names an already decoded
    position, sequence 2 with an out-of-range entry: the first proceeds as the oracle says, the other two are left
    untouched and report n_active = -1 (the rule an out-of-range window follows in block mode)."""
    import paper_2603_18489_b200 as ec

    B, L, prompt, window, k, n_cap = 3, 256, 100, 16, 2, 64
    dev = torch.device("cuda")
    hist, state = ec.new_history(B, L), ec.new_step_state(B, 1)
    masked_np = np.ones((B, L), np.uint8)
    masked_np[:, :prompt] = 0
    masked = torch.from_numpy(masked_np.copy()).to(dev)
    first = oracle.sliding_window_rows(masked_np[0], window).astype(np.int32)
    lists = np.full((B, n_cap), -1, np.int32)
    lists[0, :window] = first
    lists[1, :window] = first
    lists[1, 3] = 7                      # a prompt position: not masked
    lists[2, :window] = first
    lists[2, 5] = L + 4                  # out of range
    idx = torch.from_numpy(lists.copy()).to(dev)
    flags = np.zeros((B, window), np.uint8)
    flags[:, [1, 3, 5]] = 1
    dec = np.zeros(B, np.int32)
    ec.ec_select_recent_sliding(hist, state, masked, torch.from_numpy(flags.reshape(-1)).to(dev), window,
                                torch.from_numpy(dec).to(dev), k, idx)
    torch.cuda.synchronize()
    g_hist, g_state, g_idx, g_m = hist.cpu().numpy(), state.cpu().numpy(), idx.cpu().numpy(), masked.cpu().numpy()
    H, M = np.full(L, -np.inf), masked_np[0].copy()
    new_rows, skip, dt, t = oracle.sliding_step_bookkeeping(H, M, 1, 0, first.astype(np.int64), flags[0], 0, k, window)
    assert g_state[0].tolist() == [t, dt, int(skip), new_rows.size]
    assert g_idx[0, :new_rows.size].tolist() == new_rows.tolist() and np.array_equal(g_m[0], M)
    for b in (1, 2):
        assert g_state[b].tolist() == [1, 0, 0, -1]
        assert (g_hist[b] == NEVER).all() and np.array_equal(g_m[b], masked_np[b])
        assert np.array_equal(g_idx[b], lists[b])
