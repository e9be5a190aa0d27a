"""The allocation-free attention call against the context-based one.

nfd_attention_noalloc serves hosts that cannot call cudaMalloc where they need
attention (during a stream capture, in a frame loop that bans allocator calls,
under a memory arena they do not own): its only working memory is a fixed array
inside the library.  This file is collected last on purpose, so that a run that
stops at the first failure has already run every other test.  It must pass
alone in a fresh process and after the other tests, hence two calls in a row
with different shapes: the second one reuses the array the first one wrote.
"""
import numpy as np
import pytest

from paper_2506_01380_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _run_case(g, torch, n_kv, n_q, window, seed, H, T, dh):
    from paper_2506_01380_b200 import nfd as N
    q, k, v = I.make_qkv(H, dh, n_q * T, n_kv * T, seed=seed)
    tq, tk, tv = [torch.as_tensor(a).cuda().bfloat16() for a in (q, k, v)]
    ref = g.attention(tq, tk, tv, n_q, n_kv, window)                  # existing entry point
    # the allocation-free call takes frame pages [n_kv, H, T, dh]
    pages = lambda x: x.view(H, n_kv, T, dh).permute(1, 0, 2, 3).contiguous()
    out = torch.full((n_q * T, H * dh), float("nan"), device="cuda", dtype=torch.bfloat16)
    kp, vp = pages(tk), pages(tv)
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    N.attention_noalloc(tq, kp, vp, n_q, window, out)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before
    a, b = out.float().cpu().numpy().astype(np.float64), ref.float().cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(a))
    max_abs = np.abs(a - b).max()
    rel = np.linalg.norm(a - b) / np.linalg.norm(b)
    assert max_abs <= 3e-2 and rel <= 1e-2, (max_abs, rel)          # the bf16 tolerance of the parity tests


def test_noalloc_attention_matches_context_attention_twice():
    import torch
    from paper_2506_01380_b200 import nfd as N
    cfg = I.make_cfg("nfd310m", n_layers=1, ctx_frames=16, max_spec=4)
    g = N.NFD(cfg, I.make_weights(cfg, 0))
    H, T, dh = 16, 336, 64
    _run_case(g, torch, n_kv=6, n_q=2, window=3, seed=1, H=H, T=T, dh=dh)
    _run_case(g, torch, n_kv=17, n_q=1, window=16, seed=2, H=H, T=T, dh=dh)    # second call in a row, other shape
    # sizes beyond the fixed array are refused, nothing is launched
    x = torch.zeros(16, device="cuda", dtype=torch.bfloat16)
    rc = N.load().nfd_attention_noalloc(x.data_ptr(), x.data_ptr(), x.data_ptr(), 1, H, dh, T, 33, 40, 1,
                                        x.data_ptr(), None)
    assert rc == -4
