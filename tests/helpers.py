"""Test-side glue: moves workload tensors between torch and the numpy-based oracle and keeps
generated inputs away from decision boundaries (ties), where a float32 kernel and the
float64 oracle may legitimately land on different sides."""
from __future__ import annotations

import numpy as np
import torch

import oracle

MARGIN = 1e-4           # distance every decision keeps from its boundary
RTOL = {torch.bfloat16: 1e-3, torch.float32: 1e-5}   # scores / probabilities


def to_np(t: torch.Tensor) -> np.ndarray:
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.uint16).numpy()
    return t.numpy()


def oracle_verify(wl, threshold):
    return oracle.sprinter_verify(to_np(wl.hidden), to_np(wl.W1), to_np(wl.b1), to_np(wl.W2),
                                  to_np(wl.b2), threshold)


def oracle_sd(wl, **kw):
    return oracle.sd_verify(to_np(wl.p_logits), to_np(wl.q_logits), wl.V, to_np(wl.draft_tokens),
                            to_np(wl.uniforms), **kw)


def enforce_margins(wl, thresholds=(0.5,), margin=MARGIN, seed=1234):
    """Redraws, in place on the CPU workload, whatever lies within `margin` of a boundary:
    hidden vectors whose score is near a threshold, uniforms near p(x)/q(x), and draw
    uniforms near an edge of the selected CDF bin.  Returns the number of redraws."""
    assert not wl.hidden.is_cuda
    g = torch.Generator().manual_seed(seed)
    redraws = 0
    # -- verifier scores
    for _ in range(20):
        s, _, _ = oracle_verify(wl, 0.5)
        near = np.zeros_like(s, bool)
        for tau in thresholds:
            near |= np.abs(s - float(np.float32(tau))) < margin
        if not near.any():
            break
        idx = np.argwhere(near)
        for b, k in idx:
            wl.hidden[b, k] = torch.randn(wl.hidden.shape[-1], generator=g).to(wl.hidden.dtype)
        redraws += len(idx)
    else:
        raise AssertionError("could not clear the verifier margins")
    # -- accept tests: |u - p(x)/q(x)| with the unclamped ratio
    out = oracle_sd(wl)
    ratio = out["p_tok"] / out["q_tok"]
    for _ in range(20):
        u = wl.uniforms[:, :wl.K].numpy().astype(np.float64)
        near = np.abs(u - ratio) < margin
        if not near.any():
            break
        for b, k in np.argwhere(near):
            wl.uniforms[b, k] = torch.rand((), generator=g)
        redraws += int(near.sum())
    else:
        raise AssertionError("could not clear the accept-test margins")
    # -- correction / bonus draw with uniforms[b, K]
    out = oracle_sd(wl)
    P, Q = to_np(wl.p_logits), to_np(wl.q_logits)
    for b in range(wl.B):
        nb = int(out["accepted_len"][b])
        if nb < 0 or (nb == wl.K and wl.Kp == wl.K):
            continue
        for _ in range(50):
            u = float(wl.uniforms[b, wl.K])
            if nb < wl.K:
                m, _ = oracle.residual_draw_margin(P[b, nb, :wl.V], Q[b, nb, :wl.V], u)
            else:
                m, _ = oracle.softmax_draw_margin(P[b, wl.K, :wl.V], u)
            if m >= margin:
                break
            wl.uniforms[b, wl.K] = torch.rand((), generator=g)
            redraws += 1
        else:
            raise AssertionError("could not clear a draw margin")
    # -- replacement draw of the SPRINTER step: row b*Kp + first_reject[b], uniform u_replace[b]
    frs = [oracle_verify(wl, tau)[2] for tau in thresholds]
    for b in range(wl.B):
        rows = sorted({int(fr[b]) for fr in frs if fr[b] < wl.K})
        for _ in range(50):
            u = float(wl.u_replace[b])
            if all(oracle.softmax_draw_margin(P[b, r, :wl.V], u)[0] >= margin for r in rows):
                break
            wl.u_replace[b] = torch.rand((), generator=g)
            redraws += 1
        else:
            raise AssertionError("could not clear a replacement margin")
    return redraws


def slice_seqs(wl, lo, hi):
    """Sequences lo .. hi-1 of a workload as views: writes go through to the parent tensors."""
    import dataclasses
    kw = {}
    for f in dataclasses.fields(wl):
        v = getattr(wl, f.name)
        if isinstance(v, torch.Tensor) and f.name not in ("W1", "b1", "W2", "b2"):
            v = v[lo:hi]
            assert v.is_contiguous()
        kw[f.name] = v
    kw["B"] = hi - lo
    return type(wl)(**kw)


def seq_parts(wl, threads=None):
    """The batch cut into one contiguous run of sequences per host thread."""
    import os
    threads = max(1, min(threads or os.cpu_count() or 1, wl.B))
    cuts = [i * wl.B // threads for i in range(threads + 1)]
    return [slice_seqs(wl, lo, hi) for lo, hi in zip(cuts[:-1], cuts[1:]) if hi > lo]


def map_parts(parts, fn):
    """fn(index, part) for every part, one host thread each (the oracle's C calls release the
    interpreter lock, so the parts run on separate cores)."""
    from concurrent.futures import ThreadPoolExecutor
    with ThreadPoolExecutor(len(parts)) as pool:
        return list(pool.map(lambda a: fn(*a), enumerate(parts)))


def enforce_margins_parallel(wl, thresholds=(0.5,), margin=MARGIN, seed=1234, threads=None):
    """enforce_margins for full-size batches: the sequences are dealt to the host cores, every
    part is cleared in place with its own redraw stream.  Returns the number of redraws."""
    parts = seq_parts(wl, threads)
    return sum(map_parts(parts, lambda i, part: enforce_margins(part, thresholds, margin, seed + i)))


def oracle_step_parallel(wl, tau, threads=None):
    """Every output of the path from the oracle, over all sequences of a host workload:
    (sd_verify dict, scores, accept, first_reject, replacement tokens)."""
    def one(_, part):
        ref = oracle_sd(part)
        s, a, fr = oracle_verify(part, tau)
        P = to_np(part.p_logits).reshape(part.B * part.Kp, part.ldv)
        t = oracle.replace_sample(P, part.V, to_np(part.u_replace), first_reject=fr, K=part.K,
                                  seq_stride=part.Kp)
        return ref, s, a, fr, t
    res = map_parts(seq_parts(wl, threads), one)
    ref = {k: np.concatenate([r[0][k] for r in res]) for k in res[0][0]}
    return (ref,) + tuple(np.concatenate([r[j] for r in res]) for j in range(1, 5))


def to_device(wl, device="cuda"):
    import dataclasses
    kw = {}
    for f in dataclasses.fields(wl):
        v = getattr(wl, f.name)
        kw[f.name] = v.to(device) if isinstance(v, torch.Tensor) else v
    return type(wl)(**kw)


def assert_close_rel(got: torch.Tensor, want: np.ndarray, rtol: float, what: str):
    got = got.detach().cpu().double().numpy()
    err = np.abs(got - want) / np.maximum(np.abs(want), 1e-300)
    assert np.all(err <= rtol), f"{what}: max rel err {err.max():.3e} > {rtol}"


def assert_mass_close(got: torch.Tensor, want: np.ndarray, rtol: float, what: str = "residual_mass"):
    """Residual mass R = sum over {p_i > q_i} of p_i - q_i: a difference of two partial masses of
    order one, each known to the relative accuracy of the probabilities, so the error scales
    with those masses and not with R.  Relative to R where R is large, to 0.1 where it is small."""
    got = got.detach().cpu().double().numpy()
    err = np.abs(got - want) / np.maximum(np.abs(want), 0.1)
    assert np.all(err <= rtol), f"{what}: max err {err.max():.3e} (relative to max(R, 0.1)) > {rtol}"
