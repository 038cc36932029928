"""Host-side replay harness of the cached denoising loop (Algorithm 1 / Appendix A of the
paper) over synthetic tensors: decode history, recent-token selection, the
skip_flag / dt_recompute bookkeeping.  It holds no softmax, attention or entropy
arithmetic: the layer-step and the gate are passed in as callables, so the same
replay drives the CUDA path and the CPU oracle in the tests.

State per sequence (Appendix A, "Initialise"):
    H[i]          step at which generated position i was decoded, -inf before (Eq. 2)
    M             positions still masked; the window is the current block of `block` positions
    skip_flag     set by the gate: E <= tau  (Algorithm 1)
    dt            steps since the last full pass (0 right after one)
Recent set (Eq. 3): K = the k most recently decoded positions, tau_R = max(min_K H, t - dt),
R = {i : H_i >= tau_R}; the active rows of a partial step are window mask rows + R.
"""
from __future__ import annotations

import numpy as np

import ec_synth as syn


class ReplayState:
    def __init__(self, w: syn.Workload, block_no: int = 0):
        self.w = w
        self.t = 0
        self.dt = 0
        self.skip_flag = False
        self.block_start = w.prompt_len + block_no * w.block
        self.H = np.full(w.ctx_len, -np.inf)           # indexed by absolute position; prompt rows stay -inf
        self.masked = np.ones(w.block, dtype=bool)      # window rows still masked

    def recent_rows(self, k: int) -> np.ndarray:
        """Eq. 3: positions with H_i >= tau_R, tau_R = max(min over the top-k of H, t - dt)."""
        decoded = np.flatnonzero(np.isfinite(self.H))
        if k == 0 or decoded.size == 0:
            return np.empty(0, np.int32)
        order = decoded[np.argsort(-self.H[decoded], kind="stable")]
        top = order[:k]
        tau_r = max(self.H[top].min(), self.t - self.dt)
        sel = decoded[self.H[decoded] >= tau_r]
        return np.sort(sel).astype(np.int32)

    def active_rows(self, k: int) -> np.ndarray | None:
        """None on a full step (step 1, or the gate asked for a recompute); otherwise the window's
        positions followed by the recent rows outside the window."""
        if self.t == 0 or not self.skip_flag:
            return None
        window = np.arange(self.block_start, self.block_start + self.w.block, dtype=np.int32)
        rec = self.recent_rows(k)
        rec = rec[(rec < self.block_start) | (rec >= self.block_start + self.w.block)]
        return np.concatenate([window, rec]).astype(np.int32)

    def record(self, decoded_rows: np.ndarray, decision: int) -> None:
        """decode-history update with the step's own index, then the gate's verdict, then t <- t + 1 (Appendix A,
        end of the loop body).  The recent set is formed at the start of the next step from (t + 1) - (dt + 1) =
        t - dt, the value Appendix A uses when it selects right after the decode."""
        pos = self.block_start + np.flatnonzero(decoded_rows)
        self.H[pos] = self.t
        self.masked[np.flatnonzero(decoded_rows)] = False
        self.skip_flag = decision == 0
        self.dt = self.dt + 1 if self.skip_flag else 0
        self.t += 1


def step_inputs(w: syn.Workload, step: int, n_active: int, sigma_centre: float | None = None) -> dict:
    """Seeded tensors of one replay step: q/k_new/v_new for n_active rows and the block's logits."""
    B, Hq, Hkv, D = w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim
    rng = np.random.Generator(np.random.PCG64(1000 * w.cfg_id + 77 + 100000 * step))
    std = 1.0 / np.sqrt(D)
    q = rng.standard_normal((B, n_active, Hq, D), dtype=np.float32) * np.float32(std)
    kn = rng.standard_normal((B, n_active, Hkv, D), dtype=np.float32) * np.float32(std)
    vn = rng.standard_normal((B, n_active, Hkv, D), dtype=np.float32) * np.float32(std)
    if sigma_centre is None:
        lg = syn.logits_rows(w.block, w.vocab, w.dtype, cfg_id=w.cfg_id, step=step)
    else:
        lg = syn.logits_rows(w.block, w.vocab, w.dtype, cfg_id=w.cfg_id, step=step,
                             sigma_lo=max(0.25, sigma_centre - 1.5), sigma_hi=sigma_centre + 1.5)
    return dict(q=syn.encode(q, w.dtype), k_new=syn.encode(kn, w.dtype), v_new=syn.encode(vn, w.dtype),
                logits=lg["logits"])


def decoded_this_step(state: ReplayState, step: int, per_step: int) -> np.ndarray:
    """uint8 [block]: which still-masked window rows get decoded at this step (seeded choice; at least one
    while any is masked, as `decode` guarantees in Algorithm 1)."""
    rng = np.random.Generator(np.random.PCG64(555 + 100000 * step + state.w.cfg_id))
    cand = np.flatnonzero(state.masked)
    out = np.zeros(state.w.block, np.uint8)
    if cand.size:
        pick = rng.choice(cand, size=min(per_step, cand.size), replace=False)
        out[pick] = 1
    return out


def run_replay(w: syn.Workload, n_steps: int, tau: float, k: int, attend_fn, gate_fn, caches,
               sigma_centre_fn=None, forced_decisions=None, per_step: int = 4):
    """Runs n_steps of refresh -> attend -> gate.  attend_fn(q, k_new, v_new, active_idx_or_None) refreshes
    `caches` in place and returns the attention output; gate_fn(logits, flags, tau) returns
    (max_entropy, decision).  forced_decisions[s] (if not None) overrides the decision that drives step
    s + 1, so that two replays stay on the same trace when |E - tau| is inside the tolerance band.
    Returns the per-step records."""
    st = ReplayState(w)
    records = []
    for s in range(n_steps):
        idx = st.active_rows(k)
        n_active = w.ctx_len if idx is None else idx.size
        centre = None if sigma_centre_fn is None else sigma_centre_fn(s)
        t = step_inputs(w, s, n_active, centre)
        idx_b = None if idx is None else np.broadcast_to(idx, (w.batch, n_active)).copy()
        out = attend_fn(t["q"], t["k_new"], t["v_new"], idx_b)
        flags = decoded_this_step(st, s, per_step)
        if not flags.any():           # block finished: open the next one (same caches, fresh window)
            st.block_start = min(st.block_start + w.block, w.ctx_len - w.block)
            st.masked[:] = True
            flags = decoded_this_step(st, s, per_step)
        E, dec = gate_fn(t["logits"], flags, tau)
        used = dec if forced_decisions is None or forced_decisions[s] is None else forced_decisions[s]
        records.append(dict(step=s, full=idx is None, n_active=n_active, out=out, E=float(E), decision=int(dec),
                            used=int(used), idx=idx))
        st.record(flags, used)
    return records


class SlidingState:
    """Sliding-window decoding (Section 2.1 of the paper: the window advances over the sequence and keeps the number of
    masked tokens being denoised constant): the window of a step is the first `window` still-masked positions of the
    generation region, which stop being contiguous as soon as a position inside is decoded.  Same history / skip_flag /
    dt bookkeeping as ReplayState."""

    def __init__(self, w: syn.Workload, window: int):
        self.w, self.window = w, window
        self.t, self.dt, self.skip_flag = 0, 0, False
        self.H = np.full(w.ctx_len, -np.inf)
        self.masked = np.zeros(w.ctx_len, dtype=bool)
        self.masked[w.prompt_len:] = True

    def window_positions(self) -> np.ndarray:
        return np.flatnonzero(self.masked)[:self.window].astype(np.int32)

    def recent_rows(self, k: int) -> np.ndarray:
        decoded = np.flatnonzero(np.isfinite(self.H))
        if k == 0 or decoded.size == 0:
            return np.empty(0, np.int32)
        order = decoded[np.argsort(-self.H[decoded], kind="stable")]
        tau_r = max(self.H[order[:k]].min(), self.t - self.dt)
        return np.sort(decoded[self.H[decoded] >= tau_r]).astype(np.int32)

    def active_rows(self, k: int) -> np.ndarray | None:
        if self.t == 0 or not self.skip_flag:
            return None
        win = self.window_positions()
        rec = self.recent_rows(k)
        return np.concatenate([win, rec[~np.isin(rec, win)]]).astype(np.int32)

    def record(self, decoded_pos: np.ndarray, decision: int) -> None:
        self.H[decoded_pos] = self.t
        self.masked[decoded_pos] = False
        self.skip_flag = decision == 0
        self.dt = self.dt + 1 if self.skip_flag else 0
        self.t += 1


def run_replay_sliding(w: syn.Workload, window: int, n_steps: int, tau: float, k: int, attend_fn, gate_fn,
                       forced_decisions=None, per_step: int = 3):
    """The sliding-window counterpart of run_replay: the gate sees the logits rows of the window's positions (one row
    per window position, `window` rows per sequence), a seeded choice of them is decoded each step."""
    st = SlidingState(w, window)
    records = []
    for s in range(n_steps):
        win = st.window_positions()
        if win.size < window:          # the generation region is nearly finished: stop the trace
            break
        idx = st.active_rows(k)
        n_active = w.ctx_len if idx is None else idx.size
        t = step_inputs(w, s, n_active)
        idx_b = None if idx is None else np.broadcast_to(idx, (w.batch, n_active)).copy()
        out = attend_fn(t["q"], t["k_new"], t["v_new"], idx_b)
        rng = np.random.Generator(np.random.PCG64(4242 + 100000 * s + w.cfg_id))
        flags = np.zeros(window, np.uint8)
        flags[rng.choice(window, size=min(per_step, window), replace=False)] = 1
        lg = syn.logits_rows(window, w.vocab, w.dtype, cfg_id=w.cfg_id, step=s)["logits"]
        E, dec = gate_fn(lg, flags, tau)
        used = dec if forced_decisions is None or forced_decisions[s] is None else forced_decisions[s]
        records.append(dict(step=s, full=idx is None, n_active=n_active, out=out, E=float(E), decision=int(dec),
                            used=int(used), idx=idx))
        st.record(win[flags != 0], used)
    return records
