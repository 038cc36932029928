"""CPU oracle for the EntropyCache hot path (fp64) -- TEST INFRASTRUCTURE ONLY.

Thin ctypes/numpy wrapper around ``ec_oracle.c``.  Only the tests, the smoke
check and the benchmark's CPU-baseline leg may import this package; the CUDA
library and its Python binding never do, and this package imports neither of
them.  Arrays are numpy arrays in storage encoding: float32, or uint16 holding
bf16 bit patterns (dtype 0 / 1).

Passages followed: Section 4.2 and Appendix A (partial step: refresh the active
rows' K/V, attend from the active rows over every position), Eq. 1 and
Algorithm 1 (entropy of each decoded row, maximum, comparison with tau), Eq. 2-3 and
Appendix A (decode history, recent-token selection, skip_flag / dt bookkeeping; plain
numpy at the end of this file).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ec_oracle.c")
_SO = os.path.join(_HERE, "libec_oracle.so")
_lib = None

F32, BF16 = 0, 1
SKIP, RECOMPUTE = 0, 1


def build(force: bool = False) -> str:
    """Compile ec_oracle.c with gcc (-O2, OpenMP) into libec_oracle.so beside it."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_SO)
        vp, i32, i64, f64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_double
        lib.oracle_kv_refresh.argtypes = [i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, i32]
        lib.oracle_kv_refresh.restype = i32
        lib.oracle_attend.argtypes = [i32, i32, i32, i32, i32, i32, f64, vp, vp, vp, i32, vp, i32, vp]
        lib.oracle_attend.restype = i32
        lib.oracle_entropy_gate.argtypes = [vp, i32, i32, i32, i64, i32, vp, ctypes.c_float,
                                            vp, vp, vp, vp, vp, vp]
        lib.oracle_entropy_gate.restype = i32
        lib.oracle_num_threads.restype = i32
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _storage(a: np.ndarray, dtype: int) -> np.ndarray:
    want = np.float32 if dtype == F32 else np.uint16
    if a.dtype != want or not a.flags.c_contiguous:
        raise TypeError(f"expected contiguous {want.__name__} storage array, got {a.dtype}")
    return a


def kv_refresh(k_cache: np.ndarray, v_cache: np.ndarray, k_new: np.ndarray, v_new: np.ndarray,
               active_idx: np.ndarray | None, dtype: int) -> None:
    """In place: cache[b, h, idx[b, i], :] <- new[b, i, h, :] (K and V).

    k_cache/v_cache [B, H_kv, L, D]; k_new/v_new [B, n, H_kv, D]; active_idx
    int32 [B, n] or None for the identity list 0..n-1 (recompute step)."""
    for a in (k_cache, v_cache, k_new, v_new):
        _storage(a, dtype)
    B, Hkv, L, D = k_cache.shape
    n = k_new.shape[1]
    assert k_new.shape == (B, n, Hkv, D) and v_new.shape == k_new.shape and v_cache.shape == k_cache.shape
    if active_idx is not None:
        active_idx = np.ascontiguousarray(active_idx, dtype=np.int32)
        assert active_idx.shape == (B, n)
    rc = _load().oracle_kv_refresh(B, L, Hkv, D, k_cache.itemsize, _ptr(k_cache), _ptr(v_cache),
                                   _ptr(k_new), _ptr(v_new), _ptr(active_idx), n)
    if rc:
        raise ValueError("oracle_kv_refresh: index out of range")


def attend(q: np.ndarray, k_cache: np.ndarray, v_cache: np.ndarray, dtype: int, *,
           scale: float = 0.0, row_sel=None) -> np.ndarray:
    """Bidirectional attention of the active rows over the whole cache.

    q [B, n, H_q, D]; caches [B, H_kv, L, D] (already refreshed).  Returns
    float64 [B, n_sel, H_q, D]; row_sel (list of indices into 0..n-1) restricts
    the computed query rows, None computes all."""
    for a in (q, k_cache, v_cache):
        _storage(a, dtype)
    B, n, Hq, D = q.shape
    _, Hkv, L, _ = k_cache.shape
    sel = None
    rows = n
    if row_sel is not None:
        sel = np.ascontiguousarray(row_sel, dtype=np.int32)
        rows = int(sel.size)
    out = np.empty((B, rows, Hq, D), dtype=np.float64)
    rc = _load().oracle_attend(B, L, Hq, Hkv, D, dtype, float(scale), _ptr(q), _ptr(k_cache),
                               _ptr(v_cache), n, _ptr(sel), rows, _ptr(out))
    if rc:
        raise ValueError("oracle_attend: bad arguments")
    return out


def refresh_and_attend(q, k_new, v_new, k_cache, v_cache, active_idx, dtype, *, scale=0.0, row_sel=None):
    """The layer-step as the paper orders it: refresh the active rows, then attend.
    The caches are modified in place (pass copies to keep the pre-image)."""
    if k_new is not None:
        kv_refresh(k_cache, v_cache, k_new, v_new, active_idx, dtype)
    return attend(q, k_cache, v_cache, dtype, scale=scale, row_sel=row_sel)


def entropy_gate(logits: np.ndarray, dtype: int, vocab: int, decoded_flags: np.ndarray, tau: float,
                 rows_per_seq: int | None = None, want_probs: bool = False) -> dict:
    """Eq. 1 and the skip/recompute rule.

    logits: storage array [R, row_stride] with row_stride >= vocab (only the
    first `vocab` columns of each row are read).  Returns dict with argmax
    int32[R], conf f64[R], entropy f64[R] (nats), max_entropy f64[B],
    decision int32[B] (1 = recompute: E > tau; 0 = skip), probs (optional)."""
    _storage(logits, dtype)
    R, stride = logits.shape
    assert stride >= vocab
    rps = R if rows_per_seq is None else rows_per_seq
    flags = np.ascontiguousarray(decoded_flags, dtype=np.uint8)
    assert flags.shape == (R,)
    nseq = R // rps if rps else 0
    argmax = np.empty(R, np.int32)
    conf = np.empty(R, np.float64)
    ent = np.empty(R, np.float64)
    maxh = np.empty(nseq, np.float64)
    dec = np.empty(nseq, np.int32)
    probs = np.empty((R, vocab), np.float64) if want_probs else None
    rc = _load().oracle_entropy_gate(_ptr(logits), dtype, R, vocab, stride, rps, _ptr(flags),
                                     ctypes.c_float(tau), _ptr(argmax), _ptr(conf), _ptr(ent),
                                     _ptr(maxh), _ptr(dec), _ptr(probs))
    if rc:
        raise ValueError("oracle_entropy_gate: n_rows must be a multiple of rows_per_seq")
    return dict(argmax=argmax, conf=conf, entropy=ent, max_entropy=maxh, decision=dec, probs=probs)


# --------------------------------------------------------------------------- #
# Recent-token selection and the per-step bookkeeping (Eq. 2-3, Appendix A).
# Plain numpy on float64 histories with -inf for "never decoded".
# --------------------------------------------------------------------------- #
def select_recent(H: np.ndarray, k: int, t: int, dt: int) -> np.ndarray:
    """Eq. 3.  H is the decode history of Eq. 2 (H_i = step at which position i was decoded, -inf otherwise).
    K = a set of k positions with the largest sum of H, i.e. the k largest entries; tau_R = max(min over K of H,
    t - dt); returns the positions of R = {i : H_i >= tau_R} in ascending order.  With fewer than k decoded
    positions K has to contain never-decoded ones, so its minimum is -inf and tau_R = t - dt; k = 0 leaves
    the minimum over an empty set, +inf, so R is empty.  Ties at the threshold all belong to R (|R| may exceed k)."""
    H = np.asarray(H, dtype=np.float64)
    if k < 0 or k > H.size:
        raise ValueError("k must lie in [0, len(H)]")
    if k == 0:
        min_k = np.inf
    else:
        min_k = np.sort(H)[::-1][k - 1]          # the k-th largest entry = min over the top-k set
    tau_r = max(min_k, float(t - dt))
    return np.flatnonzero(H >= tau_r).astype(np.int64)


def step_bookkeeping(H: np.ndarray, t: int, dt: int, decoded_pos, decision: int, k: int):
    """Appendix A, the statements after the decode of step t, in the paper's order:
        H[D] <- t;  K, tau_R, R as in Eq. 3 (with the t and dt of THIS step);
        E <= tau  =>  skip_flag <- True,  dt <- dt + 1;   else  skip_flag <- False, dt <- 0;   t <- t + 1.
    `decision` is the gate's verdict (SKIP = 0: E <= tau, RECOMPUTE = 1).  H is updated in place.
    Returns (R, skip_flag, dt_next, t_next)."""
    H[np.asarray(decoded_pos, dtype=np.int64)] = float(t)
    R = select_recent(H, k, t, dt)
    skip_flag = decision == SKIP
    dt_next = dt + 1 if skip_flag else 0
    return R, skip_flag, dt_next, t + 1


def partial_step_rows(window_start: int, block: int, R: np.ndarray) -> np.ndarray:
    """Active rows of a partial step: the positions of the current block (the mask tokens' block), then the
    recent positions outside it, ascending.  (Appendix A: the rows M u R of the partial branch; the block is
    taken whole, which keeps the row count of a step fixed at block + |R outside the block|.)"""
    window = np.arange(window_start, window_start + block, dtype=np.int64)
    R = np.asarray(R, dtype=np.int64)
    outside = R[(R < window_start) | (R >= window_start + block)]
    return np.concatenate([window, np.sort(outside)])


# --------------------------------------------------------------------------- #
# Confidence-based parallel decoding behind the gate (Section 2.1; Section 5.1: threshold 0.9).
# --------------------------------------------------------------------------- #
def decode_confident(conf: np.ndarray, masked: np.ndarray, threshold: float) -> np.ndarray:
    """Which rows of one sequence get decoded in this step: every still-masked row whose confidence (the
    probability of its most likely token) exceeds `threshold`; when no masked row does, the masked row of the
    highest confidence alone (the smallest index on ties), so that a step decodes at least one token while any is
    masked.  The comparison is made on float32 values, the precision in which the confidences are produced and
    the threshold is given.  Returns uint8 flags."""
    c = np.asarray(conf, dtype=np.float64).astype(np.float32)
    m = np.asarray(masked).astype(bool)
    flags = m & (c > np.float32(threshold))
    if not flags.any() and m.any():
        cand = np.flatnonzero(m)
        flags[cand[np.argmax(c[cand])]] = True          # argmax returns the first maximum: smallest index on ties
    return flags.astype(np.uint8)


def entropy_gate_decode(logits: np.ndarray, dtype: int, vocab: int, masked: np.ndarray, conf_threshold: float,
                        tau: float, rows_per_seq: int) -> dict:
    """Eq. 1 with the set D of newly decoded rows produced by the step itself: per-row statistics as in
    entropy_gate, D from decode_confident per sequence, then E = max entropy over D and the comparison with tau.
    Returns the statistics, `decoded` (uint8 per row), `masked_next` (masked minus decoded), `tokens` (argmax of
    the decoded rows, -1 elsewhere), `max_entropy` and `decision` per sequence."""
    masked = np.asarray(masked).astype(np.uint8)
    stats = entropy_gate(logits, dtype, vocab, np.zeros(masked.size, np.uint8), tau, rows_per_seq)
    decoded = np.zeros(masked.size, np.uint8)
    for s0 in range(0, masked.size, rows_per_seq):
        sl = slice(s0, s0 + rows_per_seq)
        decoded[sl] = decode_confident(stats["conf"][sl], masked[sl], conf_threshold)
    n_seq = masked.size // rows_per_seq
    max_h = np.full(n_seq, -np.inf)
    for b in range(n_seq):
        sl = slice(b * rows_per_seq, (b + 1) * rows_per_seq)
        h = stats["entropy"][sl][decoded[sl] != 0]
        if h.size:
            max_h[b] = h.max()
    decision = (max_h > float(np.float32(tau))).astype(np.int32)
    tokens = np.where(decoded != 0, stats["argmax"], -1).astype(np.int64)
    return dict(argmax=stats["argmax"], conf=stats["conf"], entropy=stats["entropy"], decoded=decoded,
                masked_next=(masked & (1 - decoded)).astype(np.uint8), tokens=tokens, max_entropy=max_h,
                decision=decision)


# --------------------------------------------------------------------------- #
# The three candidate gate metrics of Section 5.3 ("Choice of Thresholding Variable").
# --------------------------------------------------------------------------- #
def gate_metrics(entropy: np.ndarray, conf: np.ndarray, decoded_flags: np.ndarray, rows_per_seq: int) -> dict:
    """Per sequence, over its newly decoded rows D: (1) max entropy = max_{i in D} e(p_i), the metric of Eq. 1;
    (2) entropy sum = sum_{i in D} e(p_i); (3) max confidence = max_{i in D} max_j p_ij.  An empty D gives -inf, 0
    and -inf.  Inputs are the per-row entropies and confidences of entropy_gate."""
    e = np.asarray(entropy, dtype=np.float64)
    c = np.asarray(conf, dtype=np.float64)
    f = np.asarray(decoded_flags).astype(bool)
    n_seq = e.size // rows_per_seq
    out = dict(max_entropy=np.full(n_seq, -np.inf), entropy_sum=np.zeros(n_seq), max_conf=np.full(n_seq, -np.inf))
    for b in range(n_seq):
        sl = slice(b * rows_per_seq, (b + 1) * rows_per_seq)
        d = f[sl]
        if d.any():
            out["max_entropy"][b] = e[sl][d].max()
            out["entropy_sum"][b] = e[sl][d].sum()
            out["max_conf"][b] = c[sl][d].max()
    return out


# --------------------------------------------------------------------------- #
# Sliding-window decoding (Section 2.1; the paper's evaluation mode, window size 32).
# --------------------------------------------------------------------------- #
def sliding_window_rows(masked: np.ndarray, window: int) -> np.ndarray:
    """The window of a step: the first `window` still-masked positions, ascending (fewer when fewer remain), so
    that the number of masked tokens being denoised stays constant while the window advances over the sequence."""
    return np.flatnonzero(np.asarray(masked) != 0)[:window].astype(np.int64)


def sliding_step_bookkeeping(H: np.ndarray, masked: np.ndarray, t: int, dt: int, window_rows: np.ndarray,
                             decoded_flags: np.ndarray, decision: int, k: int, window: int):
    """Appendix A's statements after the decode of step t, with the mask tokens M given by a sliding window:
    the flagged rows of the current window are decoded (H <- t, mask cleared), R follows Eq. 3, then skip_flag / dt / t,
    then the next window.  H and masked are updated in place.  Returns (rows of the next partial step = next window
    followed by R ascending, skip_flag, dt_next, t_next); the window and R are disjoint because R holds decoded
    positions only."""
    pos = np.asarray(window_rows, dtype=np.int64)[np.asarray(decoded_flags)[:len(window_rows)] != 0]
    masked[pos] = 0
    R, skip_flag, dt_next, t_next = step_bookkeeping(H, t, dt, pos, decision, k)
    nxt = sliding_window_rows(masked, window)
    return np.concatenate([nxt, R]), skip_flag, dt_next, t_next
