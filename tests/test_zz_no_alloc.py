"""The allocation-free attention call against the context-based one and the oracle.

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

from oracle import nfd_oracle as O
from paper_2506_01380_b200 import inputs as I

pytestmark = pytest.mark.gpu

TOL = {"bf16": (3e-2, 1e-2), "fp32": (1e-4, 1e-4)}       # the tolerances of the parity tests


def _close(a, b, kind, what):
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    assert np.all(np.isfinite(a)), what
    max_abs = np.abs(a - b).max()
    rel = np.linalg.norm(a - b) / np.linalg.norm(b)
    assert max_abs <= TOL[kind][0] and rel <= TOL[kind][1], (what, max_abs, rel)


def _run_case(torch, kind, n_kv, n_q, window, seed, H, T, dh, g=None):
    from paper_2506_01380_b200 import nfd as N
    tdt = torch.bfloat16 if kind == "bf16" else torch.float32
    q, k, v = I.make_qkv(H, dh, n_q * T, n_kv * T, seed=seed, bf16=(kind == "bf16"))
    tq, tk, tv = [torch.as_tensor(a).cuda().to(tdt) for a in (q, k, v)]
    # the allocation-free call takes frame pages [n_kv, H, T, dh]
    pages = lambda x: x.view(H, n_kv, T, dh).permute(1, 0, 2, 3).contiguous()
    out = torch.full((n_q * T, H * dh), float("nan"), device="cuda", dtype=tdt)
    kp, vp = pages(tk), pages(tv)
    N.attention_noalloc(tq, kp, vp, n_q, window, out)                 # first call on the device: symbol look-up
    out.fill_(float("nan"))
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]                        # the driver's count: sees any cudaMalloc
    N.attention_noalloc(tq, kp, vp, n_q, window, out)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before, "the call must not allocate device memory"
    got = out.float().cpu().numpy()
    qf = np.repeat(np.arange(n_kv - n_q, n_kv), T)
    kf = np.repeat(np.arange(n_kv), T)
    ref = O.attention_block_causal(q, k, v, qf, kf, window).transpose(1, 0, 2).reshape(n_q * T, H * dh)
    _close(got, ref, kind, "against the oracle")
    if g is not None:
        ctx = g.attention(tq, tk, tv, n_q, n_kv, window)              # the existing entry point
        _close(got, ctx.float().cpu().numpy(), kind, "against nfd_attention")


def test_noalloc_attention_matches_context_attention_twice():
    import torch
    from paper_2506_01380_b200 import nfd as N
    cfg = I.make_cfg("nfd310m", n_layers=1, ctx_frames=16, max_spec=4)
    g = N.NFD(cfg, I.make_weights(cfg, 0))
    H, T, dh = 16, 336, 64
    _run_case(torch, "bf16", n_kv=6, n_q=2, window=3, seed=1, H=H, T=T, dh=dh, g=g)
    _run_case(torch, "bf16", n_kv=17, n_q=1, window=16, seed=2, H=H, T=T, dh=dh, g=g)   # second call, other shape
    # sizes beyond the fixed array are refused, nothing is launched
    x = torch.zeros(16, device="cuda", dtype=torch.bfloat16)
    lib = N.load()
    rc = lib.nfd_attention_noalloc(x.data_ptr(), x.data_ptr(), x.data_ptr(), 1, H, dh, T, 33, 40, 1,
                                   x.data_ptr(), None)
    assert rc == -4
    # ... and so are sizes whose products would not fit the kernel's 32-bit indices
    for heads, tok in ((2048, 64), (16, (1 << 20) + 1), (1024, 1 << 20)):
        rc = lib.nfd_attention_noalloc(x.data_ptr(), x.data_ptr(), x.data_ptr(), 1, heads, dh, tok, 32, 40, 1,
                                       x.data_ptr(), None)
        assert rc == -4, (heads, tok, rc)


@pytest.mark.parametrize("kind,H,T,dh", [("fp32", 4, 64, 32), ("bf16", 2, 96, 128), ("fp32", 3, 40, 64)])
def test_noalloc_attention_other_types_and_head_sizes(kind, H, T, dh):
    """fp32 storage and the head dimensions 32 and 128, against the oracle (no context is involved)."""
    import torch
    _run_case(torch, kind, n_kv=5, n_q=2, window=2, seed=7, H=H, T=T, dh=dh)
    _run_case(torch, kind, n_kv=3, n_q=3, window=4, seed=8, H=H, T=T, dh=dh)
