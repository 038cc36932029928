"""Seeded synthetic inputs for the EntropyCache hot path.

This module only *draws* tensors: shapes, seeds, value distributions, storage
encodings (fp32, or bf16 carried as uint16 bit patterns) and index lists.  It
contains none of the method's arithmetic (no softmax, no entropy, no attention),
so both the CPU oracle's tests and the CUDA path's tests can feed from it
without sharing any computation.

Workload shapes follow the two model geometries the paper evaluates
(Section 5.1: LLaDA-8B-Instruct and Dream-7B-Instruct, window/block size 32)
with the context lengths and recent-token budgets of the benchmark
configurations; the values themselves are Gaussian stand-ins, not model
activations.

Seeding rule: one ``numpy.random.Generator(PCG64(seed))`` per tensor,
``seed = 1000 * config_id + tensor_id (+ 100000 * step for replays)``.
Values are drawn in fp32 on the host and then rounded once
(round-to-nearest-even) to the storage dtype, so every consumer reads the same
bits.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
import numpy as np

F32 = 0
BF16 = 1


# --------------------------------------------------------------------------- #
# storage encodings
# --------------------------------------------------------------------------- #
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even); returns uint16 bit patterns.
    +-inf are kept; NaN stays NaN."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    nan = np.isnan(x)
    rounded = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)
    out = rounded.astype(np.uint16)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to fp32."""
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def encode(x: np.ndarray, dtype: int) -> np.ndarray:
    """fp32 array -> storage array (float32, or uint16 holding bf16 bits)."""
    if dtype == F32:
        return np.ascontiguousarray(x, dtype=np.float32)
    if dtype == BF16:
        return f32_to_bf16_bits(x)
    raise ValueError(f"unknown dtype {dtype}")


def decode_f64(a: np.ndarray, dtype: int) -> np.ndarray:
    """storage array -> float64 (exact widening)."""
    if dtype == F32:
        return np.asarray(a, dtype=np.float32).astype(np.float64)
    return bf16_bits_to_f32(a).astype(np.float64)


def elem_bytes(dtype: int) -> int:
    return 4 if dtype == F32 else 2


# --------------------------------------------------------------------------- #
# workload geometry
# --------------------------------------------------------------------------- #
@dataclass(frozen=True)
class Workload:
    """Geometry of one benchmark configuration (one layer unless n_layers > 1)."""
    cfg_id: int
    name: str
    dtype: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    prompt_len: int
    gen_len: int
    block: int
    k_recent: int
    vocab: int
    n_layers: int = 1
    n_steps: int = 1

    @property
    def ctx_len(self) -> int:
        return self.prompt_len + self.gen_len

    @property
    def n_skip_rows(self) -> int:
        return self.block + self.k_recent

    @property
    def n_logit_rows(self) -> int:
        return self.batch * self.block


C1 = Workload(1, "c1_tiny_fp32", F32, 1, 4, 4, 64, 128, 128, 32, 2, 1024, n_steps=8)
C2 = Workload(2, "c2_llada_l768", BF16, 1, 32, 32, 128, 512, 256, 32, 2, 126464)
C3 = Workload(3, "c3_dream_l768", BF16, 1, 28, 4, 128, 512, 256, 32, 2, 152064)
C4 = Workload(4, "c4_llada_l2048", BF16, 1, 32, 32, 128, 1024, 1024, 32, 2, 126464, n_steps=32)
C5 = Workload(5, "c5_llada_l4096", BF16, 1, 32, 32, 128, 3072, 1024, 32, 2, 126464,
              n_layers=32, n_steps=64)
C5B8 = replace(C5, name="c5_llada_l4096_b8", batch=8)
# the second model geometry of the paper's evaluation (Dream-7B: 28 query heads on 4 kv heads) at the long contexts
C4D = Workload(6, "c4_dream_l2048", BF16, 1, 28, 4, 128, 1024, 1024, 32, 2, 152064, n_steps=32)
C5D = Workload(7, "c5_dream_l4096", BF16, 1, 28, 4, 128, 3072, 1024, 32, 2, 152064, n_layers=28, n_steps=64)
WORKLOADS = {w.name: w for w in (C1, C2, C3, C4, C5, C5B8, C4D, C5D)}
BY_ID = {1: C1, 2: C2, 3: C3, 4: C4, 5: C5}

# tensor ids for the seeding rule
T_Q, T_KNEW, T_VNEW, T_KCACHE, T_VCACHE, T_IDX, T_LOGITS, T_SIGMA, T_FLAGS = range(1, 10)


def _rng(cfg_id: int, tensor_id: int, step: int = 0, salt: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(1000 * cfg_id + tensor_id + 100000 * step + 10_000_000 * salt))


def _normal(rng: np.random.Generator, shape, std: float) -> np.ndarray:
    x = rng.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    return x


# --------------------------------------------------------------------------- #
# active rows
# --------------------------------------------------------------------------- #
def active_rows(w: Workload, block_no: int = 0, k_recent: int | None = None,
                step: int = 0, salt: int = 0, shuffle: bool = False) -> np.ndarray:
    """int32 [batch, block + k]: the block's 32 mask positions followed by k
    distinct 'recently decoded' positions drawn (seeded) from the generated
    region before the block; when the block is the first one they come from the
    tail of the prompt.  Indices are unique per sequence."""
    k = w.k_recent if k_recent is None else k_recent
    start = w.prompt_len + block_no * w.block
    assert start + w.block <= w.ctx_len
    out = np.empty((w.batch, w.block + k), dtype=np.int32)
    rng = _rng(w.cfg_id, T_IDX, step, salt)
    for b in range(w.batch):
        window = np.arange(start, start + w.block, dtype=np.int32)
        lo = max(0, start - 4 * max(k, 1) - 8)
        pool = np.arange(lo, start, dtype=np.int32)
        recent = rng.choice(pool, size=k, replace=False).astype(np.int32) if k else np.empty(0, np.int32)
        row = np.concatenate([window, recent])
        if shuffle:
            rng.shuffle(row)
        out[b] = row
    return out


def consecutive_runs(seq_ids) -> list[tuple[int, int]]:
    """Maximal runs of consecutive sequence numbers in an ascending list, as (first, count) pairs:
    [0, 1, 4] -> [(0, 2), (4, 1)].  A step in which the sequences of a batch took different decisions issues one
    call per run of each kind (a run is a contiguous slice of every batch-major tensor)."""
    runs = []
    for b in seq_ids:
        if runs and runs[-1][0] + runs[-1][1] == b:
            runs[-1] = (runs[-1][0], runs[-1][1] + 1)
        else:
            runs.append((int(b), 1))
    return runs


# --------------------------------------------------------------------------- #
# attention tensors
# --------------------------------------------------------------------------- #
def attn_inputs(w: Workload, n_active: int, *, step: int = 0, salt: int = 0,
                std_qk: float | None = None, std_v: float | None = None,
                identity_idx: bool | None = None, block_no: int = 0,
                k_recent: int | None = None, shuffle_idx: bool = False,
                active_idx: np.ndarray | None = None) -> dict:
    """Draws q, k_new, v_new (for the active rows) and the K/V caches.

    Layouts (all contiguous, storage dtype of the workload):
      q, out        [batch, n_active, n_q_heads, head_dim]
      k_new, v_new  [batch, n_active, n_kv_heads, head_dim]
      k_cache, v_cache [batch, n_kv_heads, ctx_len, head_dim]
      active_idx    int32 [batch, n_active]  (None for the identity / recompute case)

    Default value law: N(0,1)/sqrt(head_dim) for q, k, v, as in the benchmark
    configurations; std_qk / std_v override it for the parity-only stress cases
    (larger std_qk makes the softmax peaky).
    """
    D = w.head_dim
    base = 1.0 / np.sqrt(D)
    sqk = base if std_qk is None else std_qk
    sv = base if std_v is None else std_v
    B, L, Hq, Hkv = w.batch, w.ctx_len, w.n_q_heads, w.n_kv_heads
    if identity_idx is None:
        identity_idx = (n_active == L) and active_idx is None
    q = _normal(_rng(w.cfg_id, T_Q, step, salt), (B, n_active, Hq, D), sqk)
    k_new = _normal(_rng(w.cfg_id, T_KNEW, step, salt), (B, n_active, Hkv, D), sqk)
    v_new = _normal(_rng(w.cfg_id, T_VNEW, step, salt), (B, n_active, Hkv, D), sv)
    k_cache = _normal(_rng(w.cfg_id, T_KCACHE, step, salt), (B, Hkv, L, D), sqk)
    v_cache = _normal(_rng(w.cfg_id, T_VCACHE, step, salt), (B, Hkv, L, D), sv)
    if active_idx is not None:
        idx = np.ascontiguousarray(active_idx, dtype=np.int32)
        assert idx.shape == (B, n_active)
    elif identity_idx:
        assert n_active == L
        idx = None
    else:
        k = (n_active - w.block) if k_recent is None else k_recent
        assert k >= 0 and w.block + k == n_active, "n_active must be block + k"
        idx = active_rows(w, block_no, k, step, salt, shuffle_idx)
    return dict(
        q=encode(q, w.dtype), k_new=encode(k_new, w.dtype), v_new=encode(v_new, w.dtype),
        k_cache=encode(k_cache, w.dtype), v_cache=encode(v_cache, w.dtype),
        active_idx=idx, n_active=n_active, dtype=w.dtype,
    )


def small_attn_workload(dtype: int, batch: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                        ctx_len: int, block: int = 4, cfg_id: int = 90) -> Workload:
    """Geometry for tiny / adversarial parity cases (not a benchmark configuration)."""
    prompt = max(ctx_len - 2 * block, 0)
    return Workload(cfg_id, f"small_{cfg_id}", dtype, batch, n_q_heads, n_kv_heads, head_dim,
                    prompt, ctx_len - prompt, block, 0, 64)


def arbitrary_active_idx(batch: int, ctx_len: int, n_active: int, seed: int) -> np.ndarray:
    """int32 [batch, n_active] unique positions per sequence in random order."""
    rng = np.random.Generator(np.random.PCG64(seed))
    out = np.empty((batch, n_active), dtype=np.int32)
    for b in range(batch):
        out[b] = rng.permutation(ctx_len)[:n_active].astype(np.int32)
    return out


# --------------------------------------------------------------------------- #
# logits
# --------------------------------------------------------------------------- #
def logits_rows(n_rows: int, vocab: int, dtype: int, *, cfg_id: int = 0, step: int = 0, salt: int = 0,
                sigma_lo: float = 0.5, sigma_hi: float = 8.0, row_stride: int | None = None) -> dict:
    """[n_rows, vocab] logits, row r ~ N(0, sigma_r^2), sigma_r ~ U(sigma_lo, sigma_hi).

    Returns the storage array with shape [n_rows, row_stride] (row_stride >= vocab;
    padding columns hold a large positive canary value that must never be read),
    the per-row sigma, and the vocab."""
    sig = _rng(cfg_id, T_SIGMA, step, salt).uniform(sigma_lo, sigma_hi, size=n_rows).astype(np.float32)
    rng = _rng(cfg_id, T_LOGITS, step, salt)
    stride = vocab if row_stride is None else row_stride
    assert stride >= vocab
    x = np.full((n_rows, stride), 1.0e4, dtype=np.float32)
    for r in range(n_rows):
        x[r, :vocab] = rng.standard_normal(size=vocab, dtype=np.float32) * sig[r]
    return dict(logits=encode(x, dtype), sigma=sig, vocab=vocab, row_stride=stride, dtype=dtype)


def decoded_flags(n_rows: int, n_flagged_per_seq: int, rows_per_seq: int, *, cfg_id: int = 0,
                  step: int = 0, salt: int = 0) -> np.ndarray:
    """uint8 [n_rows]; in every sequence exactly n_flagged_per_seq rows (seeded choice) are 1."""
    assert n_rows % rows_per_seq == 0 and 0 <= n_flagged_per_seq <= rows_per_seq
    rng = _rng(cfg_id, T_FLAGS, step, salt)
    f = np.zeros(n_rows, dtype=np.uint8)
    for s in range(n_rows // rows_per_seq):
        pick = rng.choice(rows_per_seq, size=n_flagged_per_seq, replace=False)
        f[s * rows_per_seq + pick] = 1
    return f


def drifting_sigma_centre(step: int, period: int = 16, mid: float = 4.5, amp: float = 3.0) -> float:
    """Centre of the per-row sigma band at a replay step: a slow oscillation so
    that row entropies cross typical thresholds during a replay."""
    return float(mid + amp * np.sin(2.0 * np.pi * step / period))
