"""replace_sample_static: the variant for callers that may not allocate device memory (its
scratch is a fixed array inside the library).  Checked through the C ABI against
replace_sample with a caller workspace: token ids must be identical, on two calls in a row
with different inputs, because the second call finds the first call's leftovers in the shared
scratch.  Collected last on purpose (file name), so a run that stops at the first failure
has already run every other test."""
import ctypes as C

import pytest
import torch

pytestmark = pytest.mark.gpu


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _call_static(L, tl, V, u, tokens, rows=None, fr=None, K=0, seq_stride=1):
    ldv = tl.shape[-1]
    return L.replace_sample_static(_ptr(tl), ldv, V, tl.numel() // ldv, _ptr(rows), _ptr(fr), K,
                                   seq_stride, u.numel(), _ptr(u), 1 if tl.dtype == torch.bfloat16 else 0,
                                   _ptr(tokens), C.c_void_p(torch.cuda.current_stream().cuda_stream))


def test_static_scratch_matches_workspace_variant_twice():
    import paper_2502_04557_b200 as spr
    L = spr.lib()
    g = torch.Generator().manual_seed(77)
    # first call: bf16, several chunks per row with a ragged tail, gated draws
    V1, K = 20011, 3
    tl1 = (torch.randn((40 * K, V1), generator=g) * 3).to(torch.bfloat16).cuda()
    u1 = torch.rand(40, generator=g).cuda()
    fr1 = torch.randint(0, K + 1, (40,), generator=g, dtype=torch.int32).cuda()
    # second call: fp32, other sizes, explicit rows, fewer draws than the first call
    V2 = 5000
    tl2 = (torch.randn((9, V2), generator=g) * 2).cuda()
    u2 = torch.rand(7, generator=g).cuda()
    rows2 = torch.tensor([8, 0, 3, 3, 7, 1, 5], dtype=torch.int32).cuda()

    ws = spr.Workspace(max(spr.workspace_bytes(1, 40, 1, V1, 1, 0, spr.BF16),
                           spr.workspace_bytes(1, 7, 1, V2, 1, 0, spr.F32)))
    want1 = spr.replace_sample(tl1, V1, u1, ws, first_reject=fr1, K=K, seq_stride=K)
    want2 = spr.replace_sample(tl2, V2, u2, ws, rows=rows2)
    assert ws.device_status() == 0

    got1 = torch.full((40,), -5, dtype=torch.int32, device="cuda")
    got2 = torch.full((7,), -5, dtype=torch.int32, device="cuda")
    assert _call_static(L, tl1, V1, u1, got1, fr=fr1, K=K, seq_stride=K) == 0
    assert _call_static(L, tl2, V2, u2, got2, rows=rows2) == 0
    torch.cuda.synchronize()
    assert torch.equal(got1, want1)
    assert torch.equal(got2, want2)
    assert (want1[fr1 >= K] == -1).all() and (want1[fr1 < K] >= 0).all() and (want2 >= 0).all()
    # the same through the Python wrapper, a third call on the same scratch
    got3 = torch.empty_like(got1)
    spr.replace_sample_static(tl1, V1, u1, got3, first_reject=fr1, K=K, seq_stride=K)
    assert torch.equal(got3, want1)


def test_static_scratch_rejects_oversized_requests():
    import paper_2502_04557_b200 as spr
    L = spr.lib()
    tl = torch.zeros((2, 64), device="cuda")
    # more draws than the built-in scratch has tickets for
    u = torch.zeros(1025, device="cuda")
    tok = torch.zeros(1025, dtype=torch.int32, device="cuda")
    rows = torch.zeros(1025, dtype=torch.int32, device="cuda")
    assert _call_static(L, tl, 64, u, tok, rows=rows) == 3          # SPR_ERR_WORKSPACE
    # fewer draws, but too many step partials: n * ceil(V / 512) = 600 * 254 > 65536
    V = 130000
    big = torch.zeros((1, V), device="cuda")
    u = torch.zeros(600, device="cuda")
    tok = torch.zeros(600, dtype=torch.int32, device="cuda")
    rows = torch.zeros(600, dtype=torch.int32, device="cuda")
    assert _call_static(L, big, V, u, tok, rows=rows) == 3
    assert "workspace" in L.spr_status_string(3).decode()
