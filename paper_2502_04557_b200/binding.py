"""Thin ctypes binding of libsprinter: argument marshalling only.

Every function takes CUDA ``torch`` tensors (used here purely as device buffers), passes
their pointers to the C ABI declared in ``include/sprinter.h`` and returns the output
tensors.  All arithmetic happens in the CUDA kernels of the library; there is no fallback:
if the library is missing or the device is not a compute-capability-10 GPU the call raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

F32, BF16 = 0, 1
OP_SPRINTER_VERIFY, OP_REPLACE_SAMPLE, OP_SD_VERIFY, OP_SPRINTER_STEP, OP_SD_SHARD = 0, 1, 2, 3, 4
OP_VERIFIER_LABELS, OP_VERIFIER_TRAIN = 5, 6
PATH_AUTO, PATH_SIMT, PATH_TENSOR = 0, 1, 2

EXPORTS = [
    "spr_workspace_bytes", "spr_workspace_init", "sprinter_verify", "replace_sample", "sd_verify",
    "spr_device_status", "spr_status_string", "spr_last_cuda_error", "spr_version", "spr_sd_verify_launches",
    "spr_host_arena_bytes", "sprinter_verify_host", "replace_sample_host", "sd_verify_host",
    "spr_set_stage_events", "replace_sample_static", "sprinter_step", "sprinter_simulate",
    "sd_shard_stats", "sd_shard_decide", "sd_shard_weights", "sd_shard_draw", "sd_shard_decide_weights",
    "verifier_labels", "verifier_train_step", "spr_test_sprinter_verify", "spr_test_verifier_train_step",
]


class SprinterError(RuntimeError):
    def __init__(self, fn: str, status: int):
        L = lib()
        msg = L.spr_status_string(status).decode()
        if status == 4:
            msg += " (" + L.spr_last_cuda_error().decode() + ")"
        super().__init__(f"{fn}: status {status}: {msg}")
        self.status = status


_lib = None


def lib_path() -> str:
    return _build.LIB


def lib():
    """Loads libsprinter.so (never builds it implicitly on a machine without nvcc)."""
    global _lib
    if _lib is None:
        path = lib_path()
        if not os.path.exists(path):
            raise ImportError(
                f"{path} is missing: build it with `python -m paper_2502_04557_b200.build`")
        L = C.CDLL(path)
        vp, i32, i64, f32, sz = C.c_void_p, C.c_int, C.c_int64, C.c_float, C.c_size_t
        L.spr_workspace_bytes.restype = sz
        L.spr_workspace_bytes.argtypes = [i32] * 7
        L.spr_workspace_init.restype = i32
        L.spr_workspace_init.argtypes = [vp, sz, vp]
        L.sprinter_verify.restype = i32
        L.sprinter_verify.argtypes = [vp, vp, vp, vp, vp, f32, i32, i32, i32, i32, i32, i32,
                                      vp, vp, vp, vp, sz, vp]
        L.spr_test_sprinter_verify.restype = i32
        L.spr_test_sprinter_verify.argtypes = [vp, vp, vp, vp, vp, f32, i32, i32, i32, i32, i32,
                                               vp, vp, vp, vp, sz, vp, i32, i32, i32, i32, i32, C.c_uint]
        L.sprinter_step.restype = i32
        L.sprinter_step.argtypes = [vp, vp, vp, vp, vp, f32, i32, i32, i32, i32, vp, i64, i32, i32, vp,
                                    i32, i32, vp, vp, vp, vp, vp, sz, vp]
        L.sprinter_simulate.restype = i32
        L.sprinter_simulate.argtypes = [C.c_uint64, i64, i64, i32, f32, f32, i32, vp, vp, vp]
        L.replace_sample.restype = i32
        L.replace_sample.argtypes = [vp, i64, i32, i64, vp, vp, i32, i32, i32, vp, i32, vp, vp, sz, vp]
        L.sd_verify.restype = i32
        L.sd_verify.argtypes = [vp, vp, i64, vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp,
                                vp, sz, vp]
        L.sd_shard_stats.restype = i32
        L.sd_shard_stats.argtypes = [vp, vp, i64, i32, i32, vp, i32, i32, i32, i32, vp, vp, sz, vp]
        L.sd_shard_decide.restype = i32
        L.sd_shard_decide.argtypes = [vp, i32, vp, vp, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, sz, vp]
        L.sd_shard_weights.restype = i32
        L.sd_shard_weights.argtypes = [vp, vp, i64, i32, vp, vp, i32, i32, i32, i32, vp, vp, sz, vp]
        L.sd_shard_decide_weights.restype = i32
        L.sd_shard_decide_weights.argtypes = [vp, vp, i64, i32, vp, i32, vp, vp, i32, i32, i32, i32, i32,
                                              vp, vp, vp, vp, vp, vp, sz, vp]
        L.sd_shard_draw.restype = i32
        L.sd_shard_draw.argtypes = [vp, vp, i64, i32, i32, vp, vp, i32, i32, vp, vp, i32, i32, i32, i32,
                                    vp, vp, vp, sz, vp]
        L.verifier_labels.restype = i32
        L.verifier_labels.argtypes = [vp, vp, i64, vp, i32, i32, i32, i32, i32, vp, i32, vp, vp, vp, sz, vp]
        L.verifier_train_step.restype = i32
        L.verifier_train_step.argtypes = [vp, vp, i64, i32, i32, vp, vp, vp, i32, f32, f32, f32, f32, vp, vp, sz, vp]
        L.spr_test_verifier_train_step.restype = i32
        L.spr_test_verifier_train_step.argtypes = L.verifier_train_step.argtypes + [i32, C.c_uint]
        L.spr_host_arena_bytes.restype = sz
        L.spr_host_arena_bytes.argtypes = [i32, i32, i32, i32, i64, i32, i32, i32]
        L.sprinter_verify_host.restype = i32
        L.sprinter_verify_host.argtypes = [vp, vp, vp, vp, vp, f32, i32, i32, i32, i32, i32, i32,
                                           vp, vp, vp, vp, sz, vp, sz, vp]
        L.replace_sample_host.restype = i32
        L.replace_sample_host.argtypes = [vp, i64, i32, i64, vp, vp, i32, i32, i32, vp, i32, vp,
                                          vp, sz, vp, sz, vp]
        L.sd_verify_host.restype = i32
        L.sd_verify_host.argtypes = [vp, vp, i64, vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp,
                                     vp, vp, sz, vp, sz, vp]
        L.replace_sample_static.restype = i32
        L.replace_sample_static.argtypes = [vp, i64, i32, i64, vp, vp, i32, i32, i32, vp, i32, vp, vp]
        L.spr_set_stage_events.restype = None
        L.spr_set_stage_events.argtypes = [vp, vp]
        L.spr_device_status.restype = i32
        L.spr_device_status.argtypes = [vp, vp]
        L.spr_status_string.restype = C.c_char_p
        L.spr_status_string.argtypes = [i32]
        L.spr_last_cuda_error.restype = C.c_char_p
        L.spr_last_cuda_error.argtypes = []
        L.spr_version.restype = i32
        L.spr_version.argtypes = []
        L.spr_sd_verify_launches.restype = i32
        L.spr_sd_verify_launches.argtypes = [i32, i32, i32, i32]
        _lib = L
    return _lib


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported element type {t.dtype}")


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(fn: str, rc: int):
    if rc != 0:
        raise SprinterError(fn, rc)


def _dev(t: torch.Tensor, dtype=None, name="tensor"):
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}")
    return t


def _selectors(rows, first_reject, n: int):
    """The optional int32 [n] row selectors of a replacement draw: the kernel reads n entries of
    each, as 32-bit integers, so anything else is refused here."""
    for name, t in (("rows", rows), ("first_reject", first_reject)):
        if t is None:
            continue
        if t.dtype != torch.int32:
            raise TypeError(f"{name} must be torch.int32, got {t.dtype}")
        if t.numel() != n:
            raise ValueError(f"{name} must have one entry per draw ({n}), got {t.numel()}")
        _dev(t, torch.int32, name)


def sd_verify_launches(B: int, K: int, V: int, dt: int = BF16) -> int:
    """Kernels one sd_verify call launches for this shape."""
    return int(lib().spr_sd_verify_launches(B, K, V, dt))


def workspace_bytes(op: int, B: int, K: int = 1, V: int = 1, d: int = 1, h: int = 0, dt: int = BF16) -> int:
    return int(lib().spr_workspace_bytes(op, B, K, V, d, h, dt))


class Workspace:
    """Device scratch for the library calls, cleared once at creation."""

    def __init__(self, nbytes: int, device="cuda"):
        nbytes = max(int(nbytes), 256)
        self.buf = torch.empty((nbytes + 255) // 256 * 256, dtype=torch.uint8, device=device)
        assert self.buf.data_ptr() % 256 == 0
        _check("spr_workspace_init", lib().spr_workspace_init(_ptr(self.buf), self.buf.numel(), _stream()))

    @property
    def nbytes(self) -> int:
        return self.buf.numel()

    def device_status(self) -> int:
        """Synchronises the current stream; returns and clears the sticky device status."""
        return int(lib().spr_device_status(_ptr(self.buf), _stream()))

    @classmethod
    def for_problem(cls, B: int, K: int, V: int, d: int, h: int, dt: int, device="cuda"):
        n = max(workspace_bytes(OP_SPRINTER_VERIFY, B, K, V, d, h, dt),
                workspace_bytes(OP_REPLACE_SAMPLE, B, K, V, d, h, dt),
                workspace_bytes(OP_SD_VERIFY, B, K, V, d, h, dt),
                workspace_bytes(OP_SPRINTER_STEP, B, K, V, d, h, dt))
        return cls(n, device)


def sprinter_verify(hidden, W1, b1, W2, b2, threshold: float, ws: Workspace, path: int = PATH_AUTO,
                    want_scores: bool = True, out=None):
    """hidden [B,K,d]; W1 [h,d], b1 [h], W2 [h], b2 [1] (or W1 [d], b1 = W2 = None).

    Returns (scores f32 [B,K] or None, accept u8 [B,K], first_reject i32 [B])."""
    _dev(hidden, name="hidden")
    B, K, d = hidden.shape
    dt = _dt(hidden)
    _dev(W1, hidden.dtype, "W1")
    h = 0 if W1.dim() == 1 else W1.shape[0]
    if W1.shape[-1] != d:
        raise ValueError("W1 inner dimension must equal d")
    _dev(b2, torch.float32, "b2")
    if h:
        _dev(b1, torch.float32, "b1")
        _dev(W2, hidden.dtype, "W2")
        if b1.numel() != h or W2.numel() != h:
            raise ValueError("b1 and W2 must have h entries")
    else:
        b1 = W2 = None
    if out is None:
        scores = torch.empty((B, K), dtype=torch.float32, device=hidden.device) if want_scores else None
        accept = torch.empty((B, K), dtype=torch.uint8, device=hidden.device)
        first_reject = torch.empty((B,), dtype=torch.int32, device=hidden.device)
    else:
        scores, accept, first_reject = out
    rc = lib().sprinter_verify(_ptr(hidden), _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2), float(threshold),
                               B, K, d, h, dt, path, _ptr(scores), _ptr(accept), _ptr(first_reject),
                               _ptr(ws.buf), ws.nbytes, _stream())
    _check("sprinter_verify", rc)
    return scores, accept, first_reject


def sprinter_verify_shaped(hidden, W1, b1, W2, b2, threshold: float, ws: Workspace, bm: int = 0, bn: int = 0,
                           splits: int = 0, cluster_n: int = 0, flags: int = 0, spin_limit: int = 0, out=None):
    """Test hook (spr_test_sprinter_verify): the tensor-core verifier with a forced launch shape."""
    _dev(hidden, torch.bfloat16, "hidden")
    B, K, d = hidden.shape
    h = W1.shape[0]
    for t, ty, nm in ((W1, torch.bfloat16, "W1"), (b1, torch.float32, "b1"), (W2, torch.bfloat16, "W2"),
                      (b2, torch.float32, "b2")):
        _dev(t, ty, nm)
    if W1.shape[-1] != d or b1.numel() != h or W2.numel() != h:
        raise ValueError("W1 must be [h, d]; b1 and W2 must have h entries")
    if out is None:
        scores = torch.empty((B, K), dtype=torch.float32, device=hidden.device)
        accept = torch.empty((B, K), dtype=torch.uint8, device=hidden.device)
        first_reject = torch.empty((B,), dtype=torch.int32, device=hidden.device)
    else:
        scores, accept, first_reject = out
    rc = lib().spr_test_sprinter_verify(_ptr(hidden), _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2), float(threshold),
                                        B, K, d, h, BF16, _ptr(scores), _ptr(accept), _ptr(first_reject),
                                        _ptr(ws.buf), ws.nbytes, _stream(), bm, bn, splits, cluster_n, flags,
                                        spin_limit)
    _check("spr_test_sprinter_verify", rc)
    return scores, accept, first_reject


def sprinter_step(hidden, W1, b1, W2, b2, threshold: float, target_logits, V: int, uniforms,
                  ws: Workspace, path: int = PATH_AUTO, want_scores: bool = True, out=None):
    """sprinter_verify followed by the gated replace_sample, as one library call.

    target_logits [B, seq_stride, ldv]; uniforms f32 [B].
    Returns (scores or None, accept u8 [B,K], first_reject i32 [B], tokens i32 [B])."""
    _dev(hidden, name="hidden")
    B, K, d = hidden.shape
    dt = _dt(hidden)
    _dev(W1, hidden.dtype, "W1")
    h = 0 if W1.dim() == 1 else W1.shape[0]
    _dev(b2, torch.float32, "b2")
    if h:
        _dev(b1, torch.float32, "b1")
        _dev(W2, hidden.dtype, "W2")
    else:
        b1 = W2 = None
    _dev(target_logits, hidden.dtype, "target_logits")
    if target_logits.dim() != 3 or target_logits.shape[0] != B:
        raise ValueError("target_logits must be [B, seq_stride, ldv]")
    seq_stride, ldv = target_logits.shape[1], target_logits.shape[2]
    _dev(uniforms, torch.float32, "uniforms")
    if uniforms.numel() != B:
        raise ValueError("uniforms must have one entry per sequence")
    if out is None:
        dev = hidden.device
        scores = torch.empty((B, K), dtype=torch.float32, device=dev) if want_scores else None
        accept = torch.empty((B, K), dtype=torch.uint8, device=dev)
        first_reject = torch.empty((B,), dtype=torch.int32, device=dev)
        tokens = torch.empty((B,), dtype=torch.int32, device=dev)
    else:
        scores, accept, first_reject, tokens = out
    rc = lib().sprinter_step(_ptr(hidden), _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2), float(threshold),
                             B, K, d, h, _ptr(target_logits), ldv, V, seq_stride, _ptr(uniforms), dt, path,
                             _ptr(scores), _ptr(accept), _ptr(first_reject), _ptr(tokens),
                             _ptr(ws.buf), ws.nbytes, _stream())
    _check("sprinter_step", rc)
    return scores, accept, first_reject, tokens


def replace_sample(target_logits, V: int, uniforms, ws: Workspace, rows=None, first_reject=None,
                   K: int = 0, seq_stride: int = 1, out=None):
    """target_logits [R, ldv] (any leading shape is flattened to rows); returns tokens i32 [n]."""
    _dev(target_logits, name="target_logits")
    ldv = target_logits.shape[-1]
    R = target_logits.numel() // ldv
    _dev(uniforms, torch.float32, "uniforms")
    n = uniforms.numel()
    _selectors(rows, first_reject, n)
    tokens = torch.empty((n,), dtype=torch.int32, device=target_logits.device) if out is None else out
    if tokens.numel() != n:
        raise ValueError("tokens must have one entry per uniform")
    rc = lib().replace_sample(_ptr(target_logits), ldv, V, R, _ptr(rows), _ptr(first_reject), K,
                              seq_stride, n, _ptr(uniforms), _dt(target_logits), _ptr(tokens),
                              _ptr(ws.buf), ws.nbytes, _stream())
    _check("replace_sample", rc)
    return tokens


def sd_verify(p_logits, q_logits, V: int, draft_tokens, uniforms, ws: Workspace, extras: bool = True,
              out=None):
    """p_logits [B,Kp,ldv], q_logits [B,K,ldv], draft_tokens i32 [B,K], uniforms f32 [B,K+1].

    Returns dict(accepted_len, correction_token[, accept, p_tok, q_tok, residual_mass])."""
    _dev(p_logits, name="p_logits")
    _dev(q_logits, p_logits.dtype, "q_logits")
    B, Kp, ldv = p_logits.shape
    K = q_logits.shape[1]
    if q_logits.shape[0] != B or q_logits.shape[2] != ldv:
        raise ValueError("p_logits and q_logits disagree in batch or row stride")
    _dev(draft_tokens, torch.int32, "draft_tokens")
    _dev(uniforms, torch.float32, "uniforms")
    if tuple(draft_tokens.shape) != (B, K) or tuple(uniforms.shape) != (B, K + 1):
        raise ValueError("draft_tokens must be [B,K] and uniforms [B,K+1]")
    dev = p_logits.device
    if out is None:
        out = dict(accepted_len=torch.empty((B,), dtype=torch.int32, device=dev),
                   correction_token=torch.empty((B,), dtype=torch.int32, device=dev))
        if extras:
            out.update(accept=torch.empty((B, K), dtype=torch.uint8, device=dev),
                       p_tok=torch.empty((B, K), dtype=torch.float32, device=dev),
                       q_tok=torch.empty((B, K), dtype=torch.float32, device=dev),
                       residual_mass=torch.empty((B,), dtype=torch.float32, device=dev))
    rc = lib().sd_verify(_ptr(p_logits), _ptr(q_logits), ldv, _ptr(draft_tokens), _ptr(uniforms),
                         B, K, Kp, V, _dt(p_logits), _ptr(out["accepted_len"]),
                         _ptr(out["correction_token"]), _ptr(out.get("accept")), _ptr(out.get("p_tok")),
                         _ptr(out.get("q_tok")), _ptr(out.get("residual_mass")),
                         _ptr(ws.buf), ws.nbytes, _stream())
    _check("sd_verify", rc)
    return out


# ---------------------------------------------------------------------------- vocabulary shards


def _shard(t: torch.Tensor, dtype=None, name="tensor"):
    """A [*, rows, Vs] view whose last dimension is dense; rows may be strided (a column slice
    of a wider tensor).  Returns the row stride in elements."""
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}")
    B, R, Vs = t.shape
    ldv = t.stride(1)
    if t.stride(2) != 1 or ldv < Vs or (B > 1 and t.stride(0) != R * ldv):
        raise ValueError(f"{name}: rows must be dense and equally spaced")
    return ldv


def sd_shard_stats(p_shard, q_shard, v0: int, draft_tokens, ws: Workspace, out=None):
    """Pass 1 of the vocabulary-sharded sd_verify: this shard's row statistics [B*Kp, 6] f32."""
    ldv = _shard(p_shard, name="p_shard")
    if _shard(q_shard, p_shard.dtype, "q_shard") != ldv:
        raise ValueError("p_shard and q_shard must have the same row stride")
    B, Kp, Vs = p_shard.shape
    K = q_shard.shape[1]
    _dev(draft_tokens, torch.int32, "draft_tokens")
    if out is None:
        out = torch.empty((B * Kp, 6), dtype=torch.float32, device=p_shard.device)
    rc = lib().sd_shard_stats(_ptr(p_shard), _ptr(q_shard), ldv, Vs, v0, _ptr(draft_tokens), B, K, Kp,
                              _dt(p_shard), _ptr(out), _ptr(ws.buf), ws.nbytes, _stream())
    _check("sd_shard_stats", rc)
    return out


def sd_shard_decide(all_stats, draft_tokens, uniforms, V: int, Vs: int, Kp: int, dt: int, ws: Workspace,
                    extras: bool = True, out=None):
    """Pass 2: all_stats [G, B*Kp, 6] (rank order) -> accepted_len (and accept, p_tok, q_tok)."""
    _dev(all_stats, torch.float32, "all_stats")
    _dev(draft_tokens, torch.int32, "draft_tokens")
    _dev(uniforms, torch.float32, "uniforms")
    B, K = draft_tokens.shape
    G = all_stats.shape[0]
    if tuple(all_stats.shape) != (G, B * Kp, 6) or tuple(uniforms.shape) != (B, K + 1):
        raise ValueError("all_stats must be [G,B*Kp,6] and uniforms [B,K+1]")
    dev = all_stats.device
    if out is None:
        out = dict(accepted_len=torch.empty((B,), dtype=torch.int32, device=dev))
        if extras:
            out.update(accept=torch.empty((B, K), dtype=torch.uint8, device=dev),
                       p_tok=torch.empty((B, K), dtype=torch.float32, device=dev),
                       q_tok=torch.empty((B, K), dtype=torch.float32, device=dev))
    rc = lib().sd_shard_decide(_ptr(all_stats), G, _ptr(draft_tokens), _ptr(uniforms), B, K, Kp, V, Vs, dt,
                               _ptr(out["accepted_len"]), _ptr(out.get("accept")), _ptr(out.get("p_tok")),
                               _ptr(out.get("q_tok")), _ptr(ws.buf), ws.nbytes, _stream())
    _check("sd_shard_decide", rc)
    return out


def sd_shard_weights(p_shard, q_shard, accepted_len, uniforms, ws: Workspace, out=None):
    """Pass 3: this shard's share [B, 2] f64 of every sequence's correction draw."""
    ldv = _shard(p_shard, name="p_shard")
    _shard(q_shard, p_shard.dtype, "q_shard")
    B, Kp, Vs = p_shard.shape
    K = q_shard.shape[1]
    _dev(accepted_len, torch.int32, "accepted_len")
    _dev(uniforms, torch.float32, "uniforms")
    if out is None:
        out = torch.empty((B, 2), dtype=torch.float64, device=p_shard.device)
    rc = lib().sd_shard_weights(_ptr(p_shard), _ptr(q_shard), ldv, Vs, _ptr(accepted_len), _ptr(uniforms),
                                B, K, Kp, _dt(p_shard), _ptr(out), _ptr(ws.buf), ws.nbytes, _stream())
    _check("sd_shard_weights", rc)
    return out


def sd_shard_decide_weights(p_shard, q_shard, all_stats, draft_tokens, uniforms, V: int, ws: Workspace,
                            extras: bool = True):
    """Passes 2 and 3 in one launch.  Returns (dict(accepted_len[, accept, p_tok, q_tok]), weights [B,2] f64)."""
    ldv = _shard(p_shard, name="p_shard")
    _shard(q_shard, p_shard.dtype, "q_shard")
    B, Kp, Vs = p_shard.shape
    K = q_shard.shape[1]
    _dev(all_stats, torch.float32, "all_stats")
    _dev(draft_tokens, torch.int32, "draft_tokens")
    _dev(uniforms, torch.float32, "uniforms")
    G = all_stats.shape[0]
    if tuple(all_stats.shape) != (G, B * Kp, 6) or tuple(uniforms.shape) != (B, K + 1) or \
            tuple(draft_tokens.shape) != (B, K):
        raise ValueError("all_stats must be [G,B*Kp,6], draft_tokens [B,K] and uniforms [B,K+1]")
    dev = p_shard.device
    out = dict(accepted_len=torch.empty((B,), dtype=torch.int32, device=dev))
    if extras:
        out.update(accept=torch.empty((B, K), dtype=torch.uint8, device=dev),
                   p_tok=torch.empty((B, K), dtype=torch.float32, device=dev),
                   q_tok=torch.empty((B, K), dtype=torch.float32, device=dev))
    weights = torch.empty((B, 2), dtype=torch.float64, device=dev)
    rc = lib().sd_shard_decide_weights(_ptr(p_shard), _ptr(q_shard), ldv, Vs, _ptr(all_stats), G, _ptr(draft_tokens),
                                       _ptr(uniforms), B, K, Kp, V, _dt(p_shard), _ptr(out["accepted_len"]),
                                       _ptr(out.get("accept")), _ptr(out.get("p_tok")), _ptr(out.get("q_tok")),
                                       _ptr(weights), _ptr(ws.buf), ws.nbytes, _stream())
    _check("sd_shard_decide_weights", rc)
    return out, weights


def sd_shard_draw(p_shard, q_shard, v0: int, all_weights, all_stats, rank: int, accepted_len, uniforms,
                  ws: Workspace, extras: bool = True, out=None):
    """Pass 4: correction_token [B] (-1 unless this shard holds the token) and residual_mass."""
    ldv = _shard(p_shard, name="p_shard")
    _shard(q_shard, p_shard.dtype, "q_shard")
    B, Kp, Vs = p_shard.shape
    K = q_shard.shape[1]
    _dev(all_weights, torch.float64, "all_weights")
    _dev(all_stats, torch.float32, "all_stats")
    G = all_weights.shape[0]
    if tuple(all_weights.shape) != (G, B, 2) or tuple(all_stats.shape) != (G, B * Kp, 6):
        raise ValueError("all_weights must be [G,B,2] and all_stats [G,B*Kp,6]")
    dev = p_shard.device
    if out is None:
        out = dict(correction_token=torch.empty((B,), dtype=torch.int32, device=dev))
        if extras:
            out["residual_mass"] = torch.empty((B,), dtype=torch.float32, device=dev)
    rc = lib().sd_shard_draw(_ptr(p_shard), _ptr(q_shard), ldv, Vs, v0, _ptr(all_weights), _ptr(all_stats),
                             G, rank, _ptr(accepted_len), _ptr(uniforms), B, K, Kp, _dt(p_shard),
                             _ptr(out["correction_token"]), _ptr(out.get("residual_mass")),
                             _ptr(ws.buf), ws.nbytes, _stream())
    _check("sd_shard_draw", rc)
    return out


# ---------------------------------------------------------------------------- fitting the verifier


def verifier_labels(p_logits, q_logits, V: int, draft_tokens, lambdas, ws: Workspace, want_ratio: bool = True):
    """p_logits [B,Kp,ldv], q_logits [B,K,ldv], draft_tokens i32 [B,K]; lambdas: up to 8 floats.

    Returns (labels u8 [len(lambdas),B,K], ratio f32 [B,K] or None) with ratio = q(x)/p(x)."""
    _dev(p_logits, name="p_logits")
    _dev(q_logits, p_logits.dtype, "q_logits")
    B, Kp, ldv = p_logits.shape
    K = q_logits.shape[1]
    _dev(draft_tokens, torch.int32, "draft_tokens")
    if q_logits.shape[0] != B or q_logits.shape[2] != ldv or tuple(draft_tokens.shape) != (B, K):
        raise ValueError("shapes of p_logits, q_logits and draft_tokens disagree")
    lam = (C.c_float * len(lambdas))(*[float(x) for x in lambdas])
    dev = p_logits.device
    labels = torch.empty((len(lambdas), B, K), dtype=torch.uint8, device=dev)
    ratio = torch.empty((B, K), dtype=torch.float32, device=dev) if want_ratio else None
    rc = lib().verifier_labels(_ptr(p_logits), _ptr(q_logits), ldv, _ptr(draft_tokens), B, K, Kp, V,
                               _dt(p_logits), C.cast(lam, C.c_void_p), len(lambdas), _ptr(labels), _ptr(ratio),
                               _ptr(ws.buf), ws.nbytes, _stream())
    _check("verifier_labels", rc)
    return labels, ratio


def verifier_train_step(hidden, labels, theta, adam_m, adam_v, t: int, lr: float, ws: Workspace,
                        beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8, loss=None,
                        test_flags: int = 0, spin_limit: int = 0):
    """One Adam step on the mean BCE loss of sigmoid(b + w.s): hidden [N,d], labels u8 [N], theta /
    adam_m / adam_v f32 [d+1] (updated in place).  Returns the loss before the step (f32 [1]).
    test_flags / spin_limit: the test hook spr_test_verifier_train_step instead of the public call."""
    _dev(hidden, name="hidden")
    N, d = hidden.shape
    _dev(labels, torch.uint8, "labels")
    for name, a in (("theta", theta), ("adam_m", adam_m), ("adam_v", adam_v)):
        _dev(a, torch.float32, name)
        if a.numel() != d + 1:
            raise ValueError(f"{name} must have d + 1 entries")
    if labels.numel() != N:
        raise ValueError("labels must have one entry per hidden state")
    if loss is None:
        loss = torch.empty((1,), dtype=torch.float32, device=hidden.device)
    if test_flags or spin_limit:
        rc = lib().spr_test_verifier_train_step(_ptr(hidden), _ptr(labels), N, d, _dt(hidden), _ptr(theta),
                                                _ptr(adam_m), _ptr(adam_v), t, lr, beta1, beta2, eps, _ptr(loss),
                                                _ptr(ws.buf), ws.nbytes, _stream(), test_flags, spin_limit)
    else:
        rc = lib().verifier_train_step(_ptr(hidden), _ptr(labels), N, d, _dt(hidden), _ptr(theta), _ptr(adam_m),
                                       _ptr(adam_v), t, lr, beta1, beta2, eps, _ptr(loss), _ptr(ws.buf), ws.nbytes,
                                       _stream())
    _check("verifier_train_step", rc)
    return loss


# ---------------------------------------------------------------------------- host buffers


def _host(t: torch.Tensor, dtype=None, name="tensor"):
    if t.is_cuda:
        raise ValueError(f"{name} must be a host tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}")
    return t


def host_arena_bytes(op: int, B: int, K: int = 1, Kp: int = 1, ldv: int = 0, d: int = 0, h: int = 0,
                     dt: int = BF16) -> int:
    return int(lib().spr_host_arena_bytes(op, B, K, Kp, ldv, d, h, dt))


class Arena:
    """Device staging memory for the host-buffer calls."""

    def __init__(self, nbytes: int, device="cuda"):
        self.buf = torch.empty((max(int(nbytes), 256) + 255) // 256 * 256, dtype=torch.uint8, device=device)

    @property
    def nbytes(self) -> int:
        return self.buf.numel()


def sprinter_verify_host(hidden, W1, b1, W2, b2, threshold: float, arena: Arena, ws: Workspace,
                         path: int = PATH_AUTO, want_scores: bool = True, out=None):
    """Host tensors in, host tensors out (pinned memory recommended); synchronises."""
    _host(hidden, name="hidden")
    B, K, d = hidden.shape
    h = 0 if W1.dim() == 1 else W1.shape[0]
    _host(W1, hidden.dtype, "W1")
    _host(b2, torch.float32, "b2")
    if h:
        _host(b1, torch.float32, "b1")
        _host(W2, hidden.dtype, "W2")
    else:
        b1 = W2 = None
    if out is None:
        scores = torch.empty((B, K), dtype=torch.float32) if want_scores else None
        accept = torch.empty((B, K), dtype=torch.uint8)
        first_reject = torch.empty((B,), dtype=torch.int32)
    else:
        scores, accept, first_reject = out
    rc = lib().sprinter_verify_host(_ptr(hidden), _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2),
                                    float(threshold), B, K, d, h, _dt(hidden), path, _ptr(scores),
                                    _ptr(accept), _ptr(first_reject), _ptr(arena.buf), arena.nbytes,
                                    _ptr(ws.buf), ws.nbytes, _stream())
    _check("sprinter_verify_host", rc)
    return scores, accept, first_reject


def replace_sample_host(target_logits, V: int, uniforms, arena: Arena, ws: Workspace, rows=None,
                        first_reject=None, K: int = 0, seq_stride: int = 1, out=None):
    _host(target_logits, name="target_logits")
    ldv = target_logits.shape[-1]
    R = target_logits.numel() // ldv
    _host(uniforms, torch.float32, "uniforms")
    n = uniforms.numel()
    if rows is not None:
        _host(rows, torch.int32, "rows")
    if first_reject is not None:
        _host(first_reject, torch.int32, "first_reject")
    tokens = torch.empty((n,), dtype=torch.int32) if out is None else out
    rc = lib().replace_sample_host(_ptr(target_logits), ldv, V, R, _ptr(rows), _ptr(first_reject), K,
                                   seq_stride, n, _ptr(uniforms), _dt(target_logits), _ptr(tokens),
                                   _ptr(arena.buf), arena.nbytes, _ptr(ws.buf), ws.nbytes, _stream())
    _check("replace_sample_host", rc)
    return tokens


def sd_verify_host(p_logits, q_logits, V: int, draft_tokens, uniforms, arena: Arena, ws: Workspace,
                   extras: bool = False, out=None):
    _host(p_logits, name="p_logits")
    _host(q_logits, p_logits.dtype, "q_logits")
    B, Kp, ldv = p_logits.shape
    K = q_logits.shape[1]
    _host(draft_tokens, torch.int32, "draft_tokens")
    _host(uniforms, torch.float32, "uniforms")
    if out is None:
        out = dict(accepted_len=torch.empty((B,), dtype=torch.int32),
                   correction_token=torch.empty((B,), dtype=torch.int32))
        if extras:
            out.update(accept=torch.empty((B, K), dtype=torch.uint8),
                       p_tok=torch.empty((B, K), dtype=torch.float32),
                       q_tok=torch.empty((B, K), dtype=torch.float32),
                       residual_mass=torch.empty((B,), dtype=torch.float32))
    rc = lib().sd_verify_host(_ptr(p_logits), _ptr(q_logits), ldv, _ptr(draft_tokens), _ptr(uniforms),
                              B, K, Kp, V, _dt(p_logits), _ptr(out["accepted_len"]),
                              _ptr(out["correction_token"]), _ptr(out.get("accept")),
                              _ptr(out.get("p_tok")), _ptr(out.get("q_tok")),
                              _ptr(out.get("residual_mass")), _ptr(arena.buf), arena.nbytes,
                              _ptr(ws.buf), ws.nbytes, _stream())
    _check("sd_verify_host", rc)
    return out


def set_stage_events(before=None, after=None):
    """torch.cuda.Event pair (created with enable_timing=True and recorded once so that the
    handles exist) that sd_verify records around its row-statistics kernel; None to stop."""
    lib().spr_set_stage_events(None if before is None else C.c_void_p(before.cuda_event),
                               None if after is None else C.c_void_p(after.cuda_event))


def replace_sample_static(target_logits, V: int, uniforms, tokens, rows=None, first_reject=None,
                          K: int = 0, seq_stride: int = 1):
    """replace_sample on the library's built-in scratch: no workspace argument, and nothing is
    allocated here either - the caller passes the output tensor `tokens` (int32 [n]).  For
    code that must not allocate device memory around the call; limited to
    n <= 1024 draws and n * steps <= 65536 (see include/sprinter.h).  Calls that may overlap
    on one GPU race on the shared scratch: keep them on one stream."""
    _dev(target_logits, name="target_logits")
    ldv = target_logits.shape[-1]
    R = target_logits.numel() // ldv
    _dev(uniforms, torch.float32, "uniforms")
    _dev(tokens, torch.int32, "tokens")
    n = uniforms.numel()
    if tokens.numel() != n:
        raise ValueError("tokens must have one entry per uniform")
    _selectors(rows, first_reject, n)
    rc = lib().replace_sample_static(_ptr(target_logits), ldv, V, R, _ptr(rows), _ptr(first_reject), K,
                                     seq_stride, n, _ptr(uniforms), _dt(target_logits), _ptr(tokens),
                                     _stream())
    _check("replace_sample_static", rc)
    return tokens


def sprinter_simulate(seed: int, runs: int, r: int, eta_tp: float, eta_fp: float, max_tokens: int,
                      first_run: int = 0, want_runs: bool = True, device="cuda"):
    """Run lengths of an i.i.d. verifier (Theorems 2 and 3).

    Returns (n_accepted int32 [runs] or None, histogram int64 [max_tokens + 1])."""
    n = torch.empty((runs,), dtype=torch.int32, device=device) if want_runs else None
    hist = torch.empty((max_tokens + 1,), dtype=torch.int64, device=device)
    rc = lib().sprinter_simulate(int(seed), int(first_run), int(runs), int(r), float(eta_tp), float(eta_fp),
                                 int(max_tokens), _ptr(n), _ptr(hist), _stream())
    _check("sprinter_simulate", rc)
    return n, hist
