"""Python binding of libentropycache (sm_100a CUDA kernels behind a C ABI).

Argument marshalling only: every step of the hot path -- K/V refresh, active-row
attention, the entropy gate -- runs in the library's kernels.  torch is used for
device memory and streams.  There is no CPU fallback: importing this package
without the built library raises.

Functions carry the names of the C entry points declared in
``include/entropycache.h``:

    ec_kv_refresh(desc, k_cache, v_cache, k_new, v_new, active_idx)
    ec_attend(desc, q, k_new, v_new, k_cache, v_cache, active_idx, ...)
    ec_entropy_gate(logits, vocab, rows_per_seq, decoded_flags, tau, ...)

(Section 4.2 / Appendix A / Eq. 1 and Algorithm 1 of the EntropyCache paper.)
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libentropycache.so")

EC_F32, EC_BF16 = 0, 1
EC_SKIP, EC_RECOMPUTE = 0, 1
EC_ATTN_CACHE_SETTLED = 1   # ec_attn_desc.flags: nothing in flight on the stream writes the caches
EC_OK = 0


class EcError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)}")


class ec_attn_desc(ctypes.Structure):
    """Mirror of the C struct ec_attn_desc."""
    _fields_ = [("batch", ctypes.c_int32), ("ctx_len", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
                ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("scale", ctypes.c_float), ("flags", ctypes.c_uint32)]


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python paper_2603_18489_b200/build.py` "
            "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    dp = ctypes.POINTER(ec_attn_desc)
    lib.ec_kv_refresh.argtypes = [dp, vp, vp, vp, vp, vp, i32, vp]
    lib.ec_kv_refresh.restype = i32
    lib.ec_attend_workspace_bytes.argtypes = [dp, i32]
    lib.ec_attend_workspace_bytes.restype = sz
    lib.ec_attend.argtypes = [dp, vp, vp, vp, vp, vp, vp, i32, vp, vp, sz, vp, vp]
    lib.ec_attend.restype = i32
    lib.ec_attend_kernel_name.argtypes = [dp, i32, i32, i32]
    lib.ec_attend_kernel_name.restype = ctypes.c_char_p
    lib.ec_entropy_gate_workspace_bytes.argtypes = [i32, i32]
    lib.ec_entropy_gate_workspace_bytes.restype = sz
    lib.ec_entropy_gate.argtypes = [vp, i32, i32, i32, i64, i32, vp, ctypes.c_float, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.ec_entropy_gate.restype = i32
    lib.ec_entropy_gate_static.argtypes = [vp, i32, i32, i32, i64, i32, vp, ctypes.c_float, vp, vp, vp, vp, vp, vp]
    lib.ec_entropy_gate_static.restype = i32
    lib.ec_entropy_gate_metrics.argtypes = [vp, i32, i32, i32, i64, i32, vp, ctypes.c_float, vp, vp, vp, vp, vp, vp, vp,
                                            vp, sz, vp]
    lib.ec_entropy_gate_metrics.restype = i32
    lib.ec_entropy_gate_decode.argtypes = [vp, i32, i32, i32, i64, i32, vp, ctypes.c_float, ctypes.c_float, vp, vp,
                                           vp, vp, vp, vp, vp, vp, sz, vp]
    lib.ec_entropy_gate_decode.restype = i32
    lib.ec_select_recent.argtypes = [vp, i32, i32, vp, vp, vp, i32, vp, i32, vp, i32, vp]
    lib.ec_select_recent.restype = i32
    lib.ec_select_recent_sliding.argtypes = [vp, i32, i32, vp, vp, vp, i32, vp, i32, vp, i32, vp]
    lib.ec_select_recent_sliding.restype = i32
    lib.ec_workspace_init.argtypes = [vp, sz, vp]
    lib.ec_workspace_init.restype = i32
    lib.ec_status_string.argtypes = [i32]
    lib.ec_status_string.restype = ctypes.c_char_p
    lib.ec_version.restype = i32
    return lib


lib = _load()


def status_string(status: int) -> str:
    return lib.ec_status_string(int(status)).decode()


def version() -> int:
    return int(lib.ec_version())


def _check(status: int, where: str) -> None:
    if status != EC_OK:
        raise EcError(status, where)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return EC_F32
    if t.dtype == torch.bfloat16:
        return EC_BF16
    raise TypeError(f"unsupported element type {t.dtype}")


def _dev(t: torch.Tensor | None, name: str):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor (the library has no host path)")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def make_desc(batch: int, ctx_len: int, n_q_heads: int, n_kv_heads: int, head_dim: int, dtype,
              scale: float = 0.0, flags: int = 0) -> ec_attn_desc:
    code = dtype if isinstance(dtype, int) else (EC_BF16 if dtype == torch.bfloat16 else EC_F32)
    return ec_attn_desc(batch, ctx_len, n_q_heads, n_kv_heads, head_dim, code, scale, flags)


def desc_from_tensors(q: torch.Tensor, k_cache: torch.Tensor, scale: float = 0.0) -> ec_attn_desc:
    B, _, Hq, D = q.shape
    _, Hkv, L, _ = k_cache.shape
    return make_desc(B, L, Hq, Hkv, D, _dtype_code(q), scale)


def new_workspace(n_bytes: int, device="cuda") -> torch.Tensor:
    """Zero-filled device workspace of at least n_bytes (16-byte aligned by the allocator)."""
    return torch.zeros(max(int(n_bytes), 16), dtype=torch.uint8, device=device)


def ec_attend_workspace_bytes(desc: ec_attn_desc, n_active: int) -> int:
    return int(lib.ec_attend_workspace_bytes(ctypes.byref(desc), int(n_active)))


def ec_attend_kernel_name(desc: ec_attn_desc, n_active: int, with_fresh_kv: bool = True,
                          with_index_list: bool = True) -> str:
    """Host-only: which kernel (and launch shape) ec_attend picks for this geometry."""
    return lib.ec_attend_kernel_name(ctypes.byref(desc), int(n_active), int(with_fresh_kv), int(with_index_list)).decode()


def ec_entropy_gate_workspace_bytes(n_rows: int, vocab: int) -> int:
    return int(lib.ec_entropy_gate_workspace_bytes(int(n_rows), int(vocab)))


def ec_workspace_init(workspace: torch.Tensor, stream=None) -> None:
    _check(lib.ec_workspace_init(_dev(workspace, "workspace"), workspace.numel() * workspace.element_size(),
                                 _stream(stream)), "ec_workspace_init")


def ec_kv_refresh(desc: ec_attn_desc, k_cache, v_cache, k_new, v_new, active_idx, stream=None) -> None:
    """k_cache[b, h, active_idx[b, i], :] = k_new[b, i, h, :] (and V), in place, asynchronously."""
    n_active = int(k_new.shape[1])
    _check(lib.ec_kv_refresh(ctypes.byref(desc), _dev(k_cache, "k_cache"), _dev(v_cache, "v_cache"),
                             _dev(k_new, "k_new"), _dev(v_new, "v_new"), _dev(active_idx, "active_idx"),
                             n_active, _stream(stream)), "ec_kv_refresh")


def ec_attend(desc: ec_attn_desc, q, k_new, v_new, k_cache, v_cache, active_idx, out=None,
              workspace=None, dev_status=None, stream=None) -> torch.Tensor:
    """Refresh the active rows (if k_new/v_new are given), then attend from the
    active rows over the whole cache.  Returns `out` [B, n_active, H_q, D]."""
    n_active = int(q.shape[1])
    if out is None:
        out = torch.empty_like(q)
    if workspace is None:
        workspace = new_workspace(ec_attend_workspace_bytes(desc, n_active), q.device)
    _check(lib.ec_attend(ctypes.byref(desc), _dev(q, "q"), _dev(k_new, "k_new"), _dev(v_new, "v_new"),
                         _dev(k_cache, "k_cache"), _dev(v_cache, "v_cache"), _dev(active_idx, "active_idx"),
                         n_active, _dev(out, "out"), _dev(workspace, "workspace"),
                         workspace.numel() * workspace.element_size(), _dev(dev_status, "dev_status"),
                         _stream(stream)), "ec_attend")
    return out


def ec_entropy_gate(logits, vocab: int, rows_per_seq: int, decoded_flags, tau: float, *,
                    argmax_out=None, conf_out=None, entropy_out=None, max_entropy_out=None,
                    decision_out=None, workspace=None, want_rows: bool = True, stream=None) -> dict:
    """One pass over logits [R, row_stride]: per-row argmax / confidence / entropy,
    per-sequence maximum entropy over the flagged rows and the skip (0) / recompute (1)
    decision.  Outputs are device tensors; nothing is synchronised."""
    if logits.dim() != 2 or not logits.is_cuda:
        raise ValueError("logits must be a 2-D CUDA tensor [n_rows, row_stride]")
    R, stride = int(logits.shape[0]), int(logits.stride(0))
    dev = logits.device
    n_seq = R // rows_per_seq if rows_per_seq > 0 else 0
    if want_rows:
        argmax_out = torch.empty(R, dtype=torch.int32, device=dev) if argmax_out is None else argmax_out
        conf_out = torch.empty(R, dtype=torch.float32, device=dev) if conf_out is None else conf_out
        entropy_out = torch.empty(R, dtype=torch.float32, device=dev) if entropy_out is None else entropy_out
    if max_entropy_out is None:
        max_entropy_out = torch.empty(n_seq, dtype=torch.float32, device=dev)
    if decision_out is None:
        decision_out = torch.empty(n_seq, dtype=torch.int32, device=dev)
    if workspace is None:
        workspace = new_workspace(ec_entropy_gate_workspace_bytes(R, vocab), dev)
    if logits.stride(1) != 1:
        raise ValueError("logits rows must be contiguous")
    _check(lib.ec_entropy_gate(ctypes.c_void_p(logits.data_ptr()), _dtype_code(logits), R, int(vocab), stride,
                               int(rows_per_seq), _dev(decoded_flags, "decoded_flags"), float(tau),
                               _dev(argmax_out, "argmax_out"), _dev(conf_out, "conf_out"),
                               _dev(entropy_out, "entropy_out"), _dev(max_entropy_out, "max_entropy_out"),
                               _dev(decision_out, "decision_out"), _dev(workspace, "workspace"),
                               workspace.numel() * workspace.element_size(), _stream(stream)), "ec_entropy_gate")
    return dict(argmax=argmax_out, conf=conf_out, entropy=entropy_out, max_entropy=max_entropy_out,
                decision=decision_out)


EC_GATE_STATIC_MAX_ROWS = 256


def ec_entropy_gate_static(logits, vocab: int, rows_per_seq: int, decoded_flags, tau: float, *,
                           max_entropy_out, decision_out, argmax_out=None, conf_out=None, entropy_out=None,
                           stream=None) -> None:
    """ec_entropy_gate for callers that cannot allocate device memory (for example a
    server whose HBM is fully pre-partitioned): the scratch is a fixed array inside the
    library, so no workspace is passed and nothing is allocated -- which is also why every
    output tensor must be supplied by the caller.  At most EC_GATE_STATIC_MAX_ROWS rows;
    calls that may overlap on the GPU share the scratch and race; the first call on a
    device should happen outside stream capture."""
    if logits.dim() != 2 or not logits.is_cuda or logits.stride(1) != 1:
        raise ValueError("logits must be a 2-D CUDA tensor with contiguous rows")
    _check(lib.ec_entropy_gate_static(ctypes.c_void_p(logits.data_ptr()), _dtype_code(logits),
                                      int(logits.shape[0]), int(vocab), int(logits.stride(0)), int(rows_per_seq),
                                      _dev(decoded_flags, "decoded_flags"), float(tau),
                                      _dev(argmax_out, "argmax_out"), _dev(conf_out, "conf_out"),
                                      _dev(entropy_out, "entropy_out"), _dev(max_entropy_out, "max_entropy_out"),
                                      _dev(decision_out, "decision_out"), _stream(stream)),
           "ec_entropy_gate_static")


EC_H_NEVER = -(2 ** 31)


def new_step_state(batch: int, t0: int = 1, device="cuda") -> torch.Tensor:
    """int32 [batch, 4] = ec_step_state per sequence: (t, dt_recompute, skip_flag, n_active)."""
    st = torch.zeros(batch, 4, dtype=torch.int32, device=device)
    st[:, 0] = t0
    return st


def new_history(batch: int, ctx_len: int, device="cuda") -> torch.Tensor:
    """int32 [batch, ctx_len] decode history (Eq. 2), every position never decoded."""
    return torch.full((batch, ctx_len), EC_H_NEVER, dtype=torch.int32, device=device)


def ec_select_recent(history, state, decoded_flags, window_start, block: int, decision, k: int, active_idx,
                     stream=None) -> None:
    """Eq. 2-3 and the bookkeeping of Appendix A after the decode of a step (argument marshalling only).
    history int32 [B, L]; state int32 [B, 4]; decoded_flags uint8 [B * block]; window_start, decision int32 [B];
    active_idx int32 [B, n_cap] (out)."""
    batch, ctx_len = history.shape
    if history.dtype != torch.int32 or state.dtype != torch.int32 or active_idx.dtype != torch.int32:
        raise TypeError("history, state and active_idx must be int32")
    if decoded_flags.dtype != torch.uint8 or window_start.dtype != torch.int32 or decision.dtype != torch.int32:
        raise TypeError("decoded_flags must be uint8, window_start and decision int32")
    if tuple(state.shape) != (batch, 4) or active_idx.shape[0] != batch or decoded_flags.numel() != batch * block:
        raise ValueError("state must be [B, 4], active_idx [B, n_cap], decoded_flags [B * block]")
    if window_start.numel() != batch or decision.numel() != batch:
        raise ValueError("window_start and decision must hold one entry per sequence")
    _check(lib.ec_select_recent(_dev(history, "history"), int(ctx_len), int(batch), _dev(state, "state"),
                                _dev(decoded_flags, "decoded_flags"), _dev(window_start, "window_start"), int(block),
                                _dev(decision, "decision"), int(k), _dev(active_idx, "active_idx"),
                                int(active_idx.shape[1]), _stream(stream)), "ec_select_recent")


def ec_entropy_gate_decode(logits, vocab: int, rows_per_seq: int, masked, conf_threshold: float, tau: float, tokens, *,
                           decoded_out=None, argmax_out=None, conf_out=None, entropy_out=None, max_entropy_out=None,
                           decision_out=None, workspace=None, want_rows: bool = True, stream=None) -> dict:
    """The gate with confidence-based parallel decoding in front of it (argument marshalling only).  `masked`
    (uint8 [R]) and `tokens` (int32 [R]) are updated in place.  Outputs are device tensors; nothing is synchronised."""
    if logits.dim() != 2:
        raise ValueError("logits must be [n_rows, row_stride]")
    n_rows, stride = logits.shape
    dev = logits.device
    n_seq = n_rows // rows_per_seq if rows_per_seq > 0 else 0
    if masked.dtype != torch.uint8 or tokens.dtype != torch.int32 or masked.numel() != n_rows or tokens.numel() != n_rows:
        raise ValueError("masked must be uint8 [n_rows], tokens int32 [n_rows]")
    if decoded_out is None:
        decoded_out = torch.empty(n_rows, dtype=torch.uint8, device=dev)
    if want_rows:
        argmax_out = torch.empty(n_rows, dtype=torch.int32, device=dev) if argmax_out is None else argmax_out
        conf_out = torch.empty(n_rows, dtype=torch.float32, device=dev) if conf_out is None else conf_out
        entropy_out = torch.empty(n_rows, dtype=torch.float32, device=dev) if entropy_out is None else entropy_out
    if max_entropy_out is None:
        max_entropy_out = torch.empty(n_seq, dtype=torch.float32, device=dev)
    if decision_out is None:
        decision_out = torch.empty(n_seq, dtype=torch.int32, device=dev)
    if workspace is None:
        workspace = new_workspace(ec_entropy_gate_workspace_bytes(n_rows, vocab), dev)
    _check(lib.ec_entropy_gate_decode(_dev(logits, "logits"), _dtype_code(logits), int(n_rows), int(vocab), int(stride),
                                      int(rows_per_seq), _dev(masked, "masked"), float(conf_threshold), float(tau),
                                      _dev(decoded_out, "decoded_out"), _dev(tokens, "tokens"),
                                      _dev(argmax_out, "argmax_out"), _dev(conf_out, "conf_out"),
                                      _dev(entropy_out, "entropy_out"), _dev(max_entropy_out, "max_entropy_out"),
                                      _dev(decision_out, "decision_out"), _dev(workspace, "workspace"),
                                      workspace.numel() * workspace.element_size(), _stream(stream)),
           "ec_entropy_gate_decode")
    return dict(argmax=argmax_out, conf=conf_out, entropy=entropy_out, decoded=decoded_out, max_entropy=max_entropy_out,
                decision=decision_out)


def ec_entropy_gate_metrics(logits, vocab: int, rows_per_seq: int, decoded_flags, tau: float, *, workspace=None,
                            stream=None) -> dict:
    """ec_entropy_gate plus the entropy sum and the maximum confidence over the decoded rows (Section 5.3 of the
    paper); argument marshalling only.  Outputs are device tensors; nothing is synchronised."""
    if logits.dim() != 2:
        raise ValueError("logits must be [n_rows, row_stride]")
    n_rows, stride = logits.shape
    dev = logits.device
    n_seq = n_rows // rows_per_seq if rows_per_seq > 0 else 0
    f32 = lambda n: torch.empty(n, dtype=torch.float32, device=dev)
    out = dict(argmax=torch.empty(n_rows, dtype=torch.int32, device=dev), conf=f32(n_rows), entropy=f32(n_rows),
               max_entropy=f32(n_seq), decision=torch.empty(n_seq, dtype=torch.int32, device=dev),
               entropy_sum=f32(n_seq), max_conf=f32(n_seq))
    if workspace is None:
        workspace = new_workspace(ec_entropy_gate_workspace_bytes(n_rows, vocab), dev)
    _check(lib.ec_entropy_gate_metrics(_dev(logits, "logits"), _dtype_code(logits), int(n_rows), int(vocab), int(stride),
                                       int(rows_per_seq), _dev(decoded_flags, "decoded_flags"), float(tau),
                                       _dev(out["argmax"], "argmax"), _dev(out["conf"], "conf"),
                                       _dev(out["entropy"], "entropy"), _dev(out["max_entropy"], "max_entropy"),
                                       _dev(out["decision"], "decision"), _dev(out["entropy_sum"], "entropy_sum"),
                                       _dev(out["max_conf"], "max_conf"), _dev(workspace, "workspace"),
                                       workspace.numel() * workspace.element_size(), _stream(stream)),
           "ec_entropy_gate_metrics")
    return out


def ec_select_recent_sliding(history, state, masked, decoded_flags, window: int, decision, k: int, active_idx,
                             stream=None) -> None:
    """ec_select_recent for sliding-window decoding (argument marshalling only).  masked uint8 [B, L] (in/out);
    active_idx int32 [B, n_cap] holds the current window in its first `window` entries on entry and the next row
    list on return."""
    batch, ctx_len = history.shape
    if history.dtype != torch.int32 or state.dtype != torch.int32 or active_idx.dtype != torch.int32:
        raise TypeError("history, state and active_idx must be int32")
    if masked.dtype != torch.uint8 or decoded_flags.dtype != torch.uint8 or decision.dtype != torch.int32:
        raise TypeError("masked and decoded_flags must be uint8, decision int32")
    if tuple(masked.shape) != (batch, ctx_len) or tuple(state.shape) != (batch, 4) or active_idx.shape[0] != batch:
        raise ValueError("masked must be [B, L], state [B, 4], active_idx [B, n_cap]")
    if decoded_flags.numel() != batch * window or decision.numel() != batch:
        raise ValueError("decoded_flags must be [B * window], decision [B]")
    _check(lib.ec_select_recent_sliding(_dev(history, "history"), int(ctx_len), int(batch), _dev(state, "state"),
                                        _dev(masked, "masked"), _dev(decoded_flags, "decoded_flags"), int(window),
                                        _dev(decision, "decision"), int(k), _dev(active_idx, "active_idx"),
                                        int(active_idx.shape[1]), _stream(stream)), "ec_select_recent_sliding")
