"""Host logic of the replay harness (Algorithm 1 / Appendix A bookkeeping), CPU only:
step 1 is always a full pass, dt_recompute resets on a full pass and grows on a skip,
Eq. 3's recent set."""
import numpy as np

import ec_synth as syn
from _replay import ReplayState, run_replay


def _state():
    return ReplayState(syn.C1)


def test_first_step_is_always_full_and_flags_follow_the_gate():
    st = _state()
    assert st.active_rows(2) is None                      # t == 0: FullPrefill
    flags = np.zeros(32, np.uint8); flags[[3, 4]] = 1
    st.record(flags, decision=0)                          # E <= tau: skip next
    assert st.skip_flag and st.dt == 1 and st.t == 1
    rows = st.active_rows(2)
    assert rows is not None and rows.size == 32           # recent rows inside the window are not repeated
    assert len(set(rows.tolist())) == rows.size
    st.record(np.zeros(32, np.uint8), decision=1)         # E > tau: recompute next
    assert not st.skip_flag and st.dt == 0
    assert st.active_rows(2) is None


def test_recent_set_follows_eq3():
    st = _state()
    p0 = st.block_start
    st.H[[p0 - 5, p0 - 4, p0 - 3]] = [1, 2, 2]            # decoded before the window (an earlier block)
    st.t, st.dt = 3, 0
    # top-2 by recency = the two rows with H = 2; tau_R = max(2, t - dt = 3) = 3: nothing qualifies
    assert st.recent_rows(2).size == 0
    st.dt = 2                                             # tau_R = max(2, 1) = 2
    assert st.recent_rows(2).tolist() == [p0 - 4, p0 - 3]
    st.dt = 3                                             # tau_R = max(min over top-3 = 1, 0) = 1 with k = 3
    assert st.recent_rows(3).tolist() == [p0 - 5, p0 - 4, p0 - 3]
    st.skip_flag = True
    rows = st.active_rows(3)
    assert rows.size == 35 and rows[:32].tolist() == list(range(p0, p0 + 32))


def test_replay_drives_both_branches_and_counts_dt():
    w = syn.C1
    calls = []

    def attend(q, kn, vn, idx):
        calls.append(None if idx is None else idx.shape[1])
        return np.zeros(1)

    seq = iter([0, 0, 1, 0, 1, 1, 0, 0])

    def gate(logits, flags, tau):
        d = next(seq)
        return (tau + 1.0 if d else tau - 1.0), d

    rec = run_replay(w, 8, 1.5, 2, attend, gate, None)
    assert calls[0] is None                               # step 1 full
    assert [r["full"] for r in rec] == [True, False, False, True, False, True, True, False]
    assert all(c is None or c >= 32 for c in calls)


def test_sliding_window_keeps_the_masked_count_constant_and_goes_non_contiguous():
    from _replay import SlidingState

    w = syn.C1
    st = SlidingState(w, 8)
    p0 = w.prompt_len
    assert st.window_positions().tolist() == list(range(p0, p0 + 8))
    st.record(np.array([p0 + 1, p0 + 4]), decision=0)
    win = st.window_positions()
    assert win.size == 8 and win.tolist() == [p0, p0 + 2, p0 + 3, p0 + 5, p0 + 6, p0 + 7, p0 + 8, p0 + 9]
    rows = st.active_rows(2)
    assert rows[:8].tolist() == win.tolist() and sorted(rows[8:].tolist()) == [p0 + 1, p0 + 4]
    assert len(set(rows.tolist())) == rows.size


def test_harness_recent_rows_agree_with_the_oracle_on_random_histories():
    """The harness carries its own statement of Eq. 3 (it drives both arms of the replays); here it is held against
    the oracle's on random decode histories: ties at the threshold, fewer decoded positions than k, k = 0, dt = 0."""
    import oracle
    from _replay import SlidingState

    rng = np.random.Generator(np.random.PCG64(2024))
    w = syn.C1
    for trial in range(300):
        st = ReplayState(w) if trial % 2 == 0 else SlidingState(w, 8)
        n_dec = int(rng.integers(0, 40))
        pos = rng.choice(np.arange(w.prompt_len, w.ctx_len), size=n_dec, replace=False)
        st.t = int(rng.integers(1, 12))
        st.H[pos] = rng.integers(0, st.t + 1, size=n_dec).astype(np.float64)     # many ties
        st.dt = int(rng.integers(0, st.t + 1))
        k = int(rng.integers(0, 9))
        want = oracle.select_recent(st.H, k, st.t, st.dt)
        assert st.recent_rows(k).tolist() == want.tolist(), (trial, k, st.t, st.dt)
