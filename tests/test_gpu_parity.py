"""GPU parity: libnfd (through its C ABI) against the fp64 oracle on the same
seeded inputs.  Tolerances: fp32 validation mode max-abs 1e-4 / rel-L2 1e-4;
bf16 max-abs 3e-2 / rel-L2 1e-2; cache counters and rollback bit-exact."""
import math

import numpy as np
import pytest

from oracle import nfd_oracle as O
from paper_2506_01380_b200 import inputs as I

pytestmark = pytest.mark.gpu

TOL = {I.DTYPE_FP32: (1e-4, 1e-4), I.DTYPE_BF16: (3e-2, 1e-2)}


def _torch():
    import torch
    return torch


def dev(a):
    torch = _torch()
    return torch.as_tensor(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def check(got, want, dtype, what="", scale_by_magnitude=False):
    """Max-abs and relative-L2 comparison.  scale_by_magnitude: the absolute bound is
    multiplied by max(1, max|want|).  Used only for cached K/V pages of free-running
    generation under the stress weights: those values reach |x| ~ 5, where one bf16
    rounding step alone is 1.6e-2, and they are computed from frames the device
    generated itself (each already within the latent tolerance)."""
    got = got.detach().float().cpu().numpy().astype(np.float64) if hasattr(got, "detach") else np.asarray(got, float)
    want = np.asarray(want, np.float64)
    assert got.shape == want.shape, (got.shape, want.shape)
    assert np.all(np.isfinite(got)), what
    max_abs = np.abs(got - want).max()
    rel = np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30)
    a, r = TOL[dtype]
    if scale_by_magnitude:
        a = a * max(1.0, float(np.abs(want).max()))
    assert max_abs <= a and rel <= r, f"{what}: max_abs={max_abs:.3e} (tol {a}), rel_l2={rel:.3e} (tol {r})"
    return max_abs, rel


def make_pair(cfg, seed=0, kind="paper", **opts):
    from paper_2506_01380_b200.nfd import NFD
    w = I.make_weights(cfg, seed, kind)
    g = NFD(cfg, w)
    for k, v in opts.items():
        g.set_option(k, v)
    return g, O.NFDOracle(cfg, w)


def prompt(cfg, g, orc, n, seed, group=1):
    x0 = I.make_latents(cfg, n, seed)
    z = I.make_latents(cfg, n, seed + 1)
    acts = I.make_actions_uniform(cfg, n, seed + 2)
    if cfg["dtype"] == I.DTYPE_BF16:
        x0, z = I.round_bf16(x0), I.round_bf16(z)
    i = 0
    while i < n:
        m = min(group, n - i)
        g.commit_frame(dev(x0[i:i + m]), acts[i:i + m], dev(z[i:i + m]))
        orc.commit_frame(x0[i:i + m].astype(np.float64), acts[i:i + m], z[i:i + m].astype(np.float64))
        i += m
    return acts


CASES = [
    ("tiny", "paper", {}),
    ("tiny", "stress", {}),
    ("tiny", "stress", {"graph": 0}),
    ("tiny_bf16", "paper", {"fast": 0}),
    ("tiny_bf16", "stress", {"fast": 0}),
    ("tiny_bf16", "paper", {}),
    ("tiny_bf16", "stress", {}),
    ("tiny_bf16", "paper", {"fuse_ln": 0}),       # in-layer adaLN as kernels of their own
    ("tiny_bf16", "stress", {"fuse_ln": 0}),
    ("tiny_gated", "stress", {}),                 # gated MLP of width 340 (padded to 344 inside)
    ("tiny_gated_bf16", "paper", {}),
    ("tiny_gated_bf16", "stress", {}),
    ("tiny_gated_bf16", "stress", {"fuse_ln": 0}),
    ("tiny_gated_bf16", "stress", {"fast": 0}),
]


@pytest.mark.parametrize("name,kind,opts", CASES)
def test_denoise_step_after_prompt(name, kind, opts):
    """The tiny model: 4 prompt frames in the cache, one denoising step for one new frame."""
    cfg = I.make_cfg(name)
    g, orc = make_pair(cfg, 0, kind, **opts)
    acts = prompt(cfg, g, orc, 4, seed=100, group=2)
    assert g.kv_state() == (4, 0, 0) == (orc.n_committed, orc.n_tentative, orc.window_first())
    x_t = I.make_latents(cfg, 1, 200)
    t = np.float32(O.fm_time(O.trig_schedule(4)[1]))
    v = g.denoise_step(dev(x_t), float(t), 5)
    v_ref = orc.denoise_step(x_t.astype(np.float64), float(t), 5)
    check(v, v_ref, cfg["dtype"], "velocity")
    for l in range(cfg["n_layers"]):
        for f in range(5):                                  # 4 cached + the scratch frame
            K, V = g.kv_read(l, f)
            Kr, Vr = orc.kv_frame(l, f)
            check(K, Kr, cfg["dtype"], f"K l{l} f{f}")
            check(V, Vr, cfg["dtype"], f"V l{l} f{f}")
    assert g.status() == 0
    assert g.launch_count() > 0


@pytest.mark.parametrize("name,opts", [("tiny", {}), ("tiny_bf16", {}), ("tiny_bf16", {"fuse_ln": 0}),
                                       ("tiny_bf16", {"fast": 0}), ("tiny_gated_bf16", {})])
def test_rmsnorm_variant(name, opts):
    """cfg.norm = 1: RMSNorm instead of LayerNorm in every adaLN (no mean removal), on every path: fp32
    validation kernels, bf16 with the norm folded into the GEMMs, bf16 with stand-alone norm kernels, bf16
    plain kernels."""
    cfg = I.make_cfg(name, norm=1)
    g, orc = make_pair(cfg, 4, "stress", **opts)
    prompt(cfg, g, orc, 3, seed=500, group=2)
    x_t = I.make_latents(cfg, 2, 510)
    if cfg["dtype"] == I.DTYPE_BF16:
        x_t = I.round_bf16(x_t)
    v = g.denoise_step(dev(x_t), 0.4375, 2)
    check(v, orc.denoise_step(x_t.astype(np.float64), 0.4375, 2), cfg["dtype"], "velocity")
    for l in range(cfg["n_layers"]):
        for f in (2, 3, 4):
            K, V = g.kv_read(l, f)
            check(K, orc.kv_frame(l, f)[0], cfg["dtype"], f"K l{l} f{f}")
            check(V, orc.kv_frame(l, f)[1], cfg["dtype"], f"V l{l} f{f}")
    assert g.status() == 0


@pytest.mark.parametrize("name", ["tiny", "tiny_bf16"])
def test_head_dim_128(name):
    """Head dimension 128 (two heads of a 256-wide model; rotary split 32/48/48): the GEMMs take the
    tensor-core path, attention the plain kernel."""
    cfg = I.make_cfg(name, d_model=256, n_heads=2, head_dim=128, d_mlp=512, rope_t=32, rope_h=48, rope_w=48)
    g, orc = make_pair(cfg, 6, "stress")
    prompt(cfg, g, orc, 5, seed=600, group=3)                 # one more frame than the window holds
    x_t = I.make_latents(cfg, 1, 610)
    if cfg["dtype"] == I.DTYPE_BF16:
        x_t = I.round_bf16(x_t)
    v = g.denoise_step(dev(x_t), 0.6, 1)
    check(v, orc.denoise_step(x_t.astype(np.float64), 0.6, 1), cfg["dtype"], "velocity")
    assert g.kv_state() == (orc.n_committed, orc.n_tentative, orc.window_first())
    assert g.status() == 0


@pytest.mark.parametrize("name,kind", [("tiny", "stress"), ("tiny_bf16", "stress")])
def test_joint_pass_equals_sequential(name, kind):
    cfg = I.make_cfg(name)
    g, orc = make_pair(cfg, 1, kind)
    prompt(cfg, g, orc, 2, seed=300)
    x_t = I.make_latents(cfg, 3, 301)
    v_joint = g.denoise_step(dev(x_t), 0.6, 2)
    check(v_joint, orc.denoise_step(x_t.astype(np.float64), 0.6, 2), cfg["dtype"], "joint")
    torch = _torch()
    for j in range(3):
        v_j = g.denoise_step(dev(x_t[j:j + 1]), 0.6, 2, offset=j)
        assert torch.equal(v_j[0], v_joint[j]), f"frame {j}: joint pass and sequential pass differ bitwise"


@pytest.mark.parametrize("name,kind,opts", [("tiny", "stress", {}), ("tiny_bf16", "stress", {}),
                                            ("tiny_bf16", "paper", {"fast": 0})])
def test_speculate_rollback_and_eviction(name, kind, opts):
    cfg = I.make_cfg(name)          # W = 4, k_max = 4
    g, orc = make_pair(cfg, 2, kind, **opts)
    g2, _ = make_pair(cfg, 2, kind, **opts)
    acts_true = [1, 1, 1, 2, 2, 3, 3, 3, 3, 3, 4]
    S = cfg["n_steps"]
    i = 0
    while i < len(acts_true) - 1:
        k = min(3, len(acts_true) - i)
        noise = np.stack([np.concatenate([I.make_noise(cfg, 1, 1, 1000 * (i + j) + s)[0] for j in range(k)])
                          for s in range(S)])
        cz = np.concatenate([I.make_latents(cfg, 1, 5000 + i + j) for j in range(k)])
        if cfg["dtype"] == I.DTYPE_BF16:
            noise, cz = I.round_bf16(noise), I.round_bf16(cz)
        x0 = g.speculate(k, acts_true[i], dev(noise), dev(cz))
        x0_ref = orc.speculate(k, acts_true[i], noise.astype(np.float64), cz.astype(np.float64))
        check(x0, x0_ref, cfg["dtype"], f"x0 at frame {i}")
        n = O.accepted_count(acts_true, i, k)
        assert g.kv_state()[1] == k
        g.rollback(n)
        orc.rollback(n)
        # a second GPU context that only ever computes the accepted prefix
        g2.speculate(n, acts_true[i], dev(noise[:, :n]), dev(cz[:n]))
        g2.rollback(n)
        assert g.kv_state() == g2.kv_state() == (orc.n_committed, orc.n_tentative, orc.window_first())
        assert g.kv_hash() == g2.kv_hash(), "cache after rollback differs from never having speculated"
        i += n
    assert g.kv_state()[0] > cfg["ctx_frames"] + cfg["max_spec"]        # the ring wrapped
    for l in range(cfg["n_layers"]):
        for f in range(orc.window_first(), orc.n_total):
            K, V = g.kv_read(l, f)
            check(K, orc.kv_frame(l, f)[0], cfg["dtype"], f"K l{l} f{f}", scale_by_magnitude=True)
            check(V, orc.kv_frame(l, f)[1], cfg["dtype"], f"V l{l} f{f}", scale_by_magnitude=True)
    assert g.status() == 0


def test_batched_streams_match_single_streams():
    cfg = I.make_cfg("tiny_bf16", n_streams=3)
    from paper_2506_01380_b200.nfd import NFD
    torch = _torch()
    w = I.make_weights(cfg, 3, "stress")
    g = NFD(cfg, w)
    orcs = [O.NFDOracle(cfg, w) for _ in range(3)]
    S, k = cfg["n_steps"], 2
    for s in range(3):
        x0 = I.round_bf16(I.make_latents(cfg, 1 + s, 40 + s))
        a = I.make_actions_uniform(cfg, 1 + s, 50 + s)
        g.commit_frame(dev(x0), a, None, stream=s)
        orcs[s].commit_frame(x0.astype(np.float64), a, None)
    noise = I.round_bf16(np.stack([I.make_noise(cfg, S, k, 60 + s) for s in range(3)], axis=1))   # [S,3,k,...]
    actions = [1, 5, 7]
    x0 = g.speculate_batched([0, 1, 2], k, actions, dev(noise))
    for s in range(3):
        ref = orcs[s].speculate(k, actions[s], noise[:, s].astype(np.float64))
        check(x0[s], ref, cfg["dtype"], f"stream {s}")
    assert [g.kv_state(s) for s in range(3)] == [(1, 2, 0), (2, 2, 0), (3, 2, 1)]
    # single-stream calls on a second context give bitwise the same frames
    g1 = NFD(cfg, w)
    for s in range(3):
        x0s = I.round_bf16(I.make_latents(cfg, 1 + s, 40 + s))
        g1.commit_frame(dev(x0s), I.make_actions_uniform(cfg, 1 + s, 50 + s), None, stream=s)
        y = g1.speculate(k, actions[s], dev(noise[:, s]), stream=s)
        assert torch.equal(y, x0[s])
        assert g1.kv_hash(s) == g.kv_hash(s)


def test_error_codes_leave_state_unchanged():
    from paper_2506_01380_b200 import nfd as N
    torch = _torch()
    cfg = I.make_cfg("tiny")
    w = I.make_weights(cfg, 0)
    for bad in (dict(n_heads=3), dict(head_dim=48, n_heads=2, d_model=96), dict(rope_t=7), dict(max_spec=0),
                dict(dtype=5), dict(sigma_d=0.0), dict(patch=3)):
        with pytest.raises(N.NfdError) as e:
            N.NFD(dict(cfg, **bad), w)
        assert e.value.code == -1
    g = N.NFD(cfg, w)
    x = dev(I.make_latents(cfg, 1, 1))
    g.commit_frame(x, [0])
    h0, s0 = g.kv_hash(), g.kv_state()
    for fn, code in [
        (lambda: g.commit_frame(x, [99]), -4),                         # action out of range
        (lambda: g.denoise_step(x, 0.5, -1), -4),
        (lambda: g.denoise_step(x, 1.5, 0), -4),                       # FM time outside [0,1]
        (lambda: g.denoise_step(x, 0.5, 0, offset=4), -4),             # offset + k > k_max
        (lambda: g.denoise_step(x, 0.5, 0, stream=1), -4),
        (lambda: g.rollback(1), -4),                                   # nothing tentative
        (lambda: g.kv_read(0, 9), -4),
        (lambda: g.lib.nfd_denoise_step(g._h, 0, None, 1, 0.5, 0, x.data_ptr()), -2),
        (lambda: g.lib.nfd_denoise_step(g._h, 0, x.data_ptr() + 4, 1, 0.5, 0, x.data_ptr()), -3),
    ]:
        try:
            r = fn()
            got = r if isinstance(r, int) else 0
        except N.NfdError as e:
            got = e.code
        assert got == code, (got, code)
        assert g.kv_state() == s0 and g.kv_hash() == h0
    noise = dev(I.make_noise(cfg, 4, 2, 3))
    g.speculate(2, 1, noise)
    with pytest.raises(N.NfdError) as e:
        g.commit_frame(x, [0])                                          # tentative frames pending
    assert e.value.code == -5
    with pytest.raises(N.NfdError) as e:
        g.speculate(2, 1, noise)
    assert e.value.code == -5
    g.rollback(0)
    assert g.kv_state() == s0 and g.kv_hash() == h0
    assert g.status() == 0
    del torch


@pytest.mark.parametrize("fast", [0, 1])
@pytest.mark.parametrize("n_kv,n_q,window", [(5, 1, 64), (17, 1, 64), (65, 1, 64), (17, 4, 16), (9, 3, 2)])
def test_attention_alone(n_kv, n_q, window, fast):
    """Attention alone: 16 heads x 64, 336-token frames, block-causal over the cache."""
    torch = _torch()
    from paper_2506_01380_b200.nfd import NFD
    cfg = I.make_cfg("nfd310m", n_layers=1, ctx_frames=64, max_spec=4)
    g = NFD(cfg, I.make_weights(cfg, 0))
    g.set_option("fast", fast)
    T, H, dh = 336, 16, 64
    q, k, v = I.make_qkv(H, dh, n_q * T, n_kv * T, seed=n_kv * 10 + n_q)
    out = g.attention(dev(q).bfloat16(), dev(k).bfloat16(), dev(v).bfloat16(), n_q, n_kv, window)
    qf = np.repeat(np.arange(n_kv - n_q, n_kv), T)
    kf = np.repeat(np.arange(n_kv), T)
    ref = O.attention_block_causal(q, k, v, qf, kf, window)            # [H, nq, dh]
    ref = ref.transpose(1, 0, 2).reshape(n_q * T, H * dh)
    check(out, ref, I.DTYPE_BF16, "attention")
    assert g.status() == 0


def _teacher_forced(cfg, kind, n_prompt, k, seed, **opts):
    g, orc = make_pair(cfg, seed, kind, **opts)
    prompt(cfg, g, orc, n_prompt, seed=700 + seed, group=4)
    x_t = I.round_bf16(I.make_latents(cfg, k, 800 + seed))
    t = float(np.float32(O.fm_time(3 * math.pi / 8)))
    v = g.denoise_step(dev(x_t), t, 3)
    v_ref = orc.denoise_step(x_t.astype(np.float64), t, 3)
    res = check(v, v_ref, cfg["dtype"], "velocity")
    L = cfg["n_layers"]
    for l in (0, L - 1):
        for f in (0, n_prompt - 1, n_prompt, n_prompt + k - 1):
            K, V = g.kv_read(l, f)
            check(K, orc.kv_frame(l, f)[0], cfg["dtype"], f"K l{l} f{f}")
            check(V, orc.kv_frame(l, f)[1], cfg["dtype"], f"V l{l} f{f}")
    assert g.status() == 0
    return res


@pytest.mark.parametrize("kind", ["paper", "stress"])
@pytest.mark.parametrize("fuse_ln", [1, 0])
def test_310m_slice_two_layers(kind, fuse_ln):
    """Two layers at model width, with the in-layer LayerNorms folded into the neighbouring GEMMs (the
    default) and as kernels of their own."""
    _teacher_forced(I.make_cfg("nfd310m_slice"), kind, n_prompt=5, k=2, seed=0, fuse_ln=fuse_ln)


@pytest.mark.parametrize("act", [0, 1])
def test_paper_310m_shape_two_layers(act):
    """The paper's own 310M row of its size table (hidden 1024, MLP 2730, 16 heads), two layers of it: an
    MLP width that is no multiple of 8, as GELU MLP and as gated MLP."""
    _teacher_forced(I.make_cfg("paper310m", n_layers=2, act=act), "stress", n_prompt=3, k=2, seed=act)


def test_paper_130m_and_774m_shapes_one_layer():
    """Hidden widths 768 (12 heads) and 1536 (24 heads) of the paper's size table, gated MLP."""
    for name in ("paper130m", "paper774m"):
        _teacher_forced(I.make_cfg(name, n_layers=1, act=1, ctx_frames=2), "paper", n_prompt=2, k=1, seed=3)


def test_310m_full_config_teacher_forced():
    """The 310M-class shape: 24 layers, 16 context frames, one denoising pass, GPU vs oracle."""
    _teacher_forced(I.make_cfg("nfd310m"), "paper", n_prompt=16, k=1, seed=0)


def test_modulation_cache_hits_evictions_and_values():
    """The adaLN modulation is kept per (FM time, action) pair: a pass that finds its pair cached must
    give bitwise the same velocity as a context that computes it afresh, also after the pair's slot was
    replaced (more distinct pairs than slots) and recomputed."""
    from paper_2506_01380_b200.nfd import NFD
    torch = _torch()
    cfg = I.make_cfg("tiny_bf16")
    w = I.make_weights(cfg, 5, "stress")
    g, orc = NFD(cfg, w), O.NFDOracle(cfg, w)
    prompt(cfg, g, orc, 2, seed=900)
    x = dev(I.round_bf16(I.make_latents(cfg, 1, 901)))
    h0, m0 = g.cond_cache_stats()
    v_first = g.denoise_step(x, 0.625, 3).clone()
    assert g.cond_cache_stats() == (h0, m0 + 1)
    v_again = g.denoise_step(x, 0.625, 3).clone()
    assert g.cond_cache_stats() == (h0 + 1, m0 + 1)
    assert torch.equal(v_first, v_again)
    check(v_first, orc.denoise_step(x.cpu().numpy().astype(np.float64), 0.625, 3), cfg["dtype"], "velocity")
    # more distinct pairs than the cache has slots: the first pair is replaced ...
    for i in range(300):
        g.denoise_step(x, float(np.float32(0.001 * (i + 1))), i % cfg["n_actions"])
    h1, m1 = g.cond_cache_stats()
    v_refill = g.denoise_step(x, 0.625, 3).clone()
    assert g.cond_cache_stats() == (h1, m1 + 1), "the pair should have been evicted and recomputed"
    assert torch.equal(v_first, v_refill)
    # ... and a failed call leaves the cache as it was
    with pytest.raises(Exception):
        g.denoise_step(x, 0.3333, 99)
    assert g.cond_cache_stats() == (h1, m1 + 1)
    assert g.status() == 0


@pytest.mark.parametrize("name,kind,n_evals", [("tiny", "stress", 18), ("tiny", "paper", 5), ("tiny_bf16", "paper", 18),
                                               ("tiny_gated_bf16", "stress", 6)])
def test_dpmpp_sampler_matches_oracle(name, kind, n_evals):
    """The undistilled sampler (DPM-Solver++ over n_evals evaluations of the Flow-Matching model): generated
    frames, counters and the tentative K/V pages against the oracle, then rollback."""
    cfg = I.make_cfg(name)
    g, orc = make_pair(cfg, 21, kind)
    prompt(cfg, g, orc, 3, seed=300, group=3)
    k = 2
    noise = I.make_latents(cfg, k, 310)
    cz = I.make_latents(cfg, k, 311)
    if cfg["dtype"] == I.DTYPE_BF16:
        noise, cz = I.round_bf16(noise), I.round_bf16(cz)
    y = g.sample_dpmpp(k, 5, dev(noise), n_evals=n_evals, ctx_noise=dev(cz))
    ref = orc.sample_dpmpp(k, 5, noise.astype(np.float64), n_evals=n_evals, ctx_noise=cz.astype(np.float64))
    check(y, ref, cfg["dtype"], "x0")
    assert g.kv_state() == (orc.n_committed, orc.n_tentative, orc.window_first())
    assert g.kv_state()[:2] == (3, k)
    for l in range(cfg["n_layers"]):
        for f in (3, 4):
            K, V = g.kv_read(l, f)
            check(K, orc.kv_frame(l, f)[0], cfg["dtype"], f"K l{l} f{f}", scale_by_magnitude=True)
            check(V, orc.kv_frame(l, f)[1], cfg["dtype"], f"V l{l} f{f}", scale_by_magnitude=True)
    g.rollback(1), orc.rollback(1)
    assert g.kv_state() == (orc.n_committed, orc.n_tentative, orc.window_first())
    assert g.kv_state()[:2] == (4, 0)
    with pytest.raises(Exception):
        g.sample_dpmpp(k, 5, dev(noise), n_evals=0)
    assert g.status() == 0


@pytest.mark.parametrize("name", ["tiny_bf16", "tiny"])
def test_warm_modulation_fills_every_schedule_pair(name):
    """nfd_warm_modulation computes the modulation of all (sampler or context time, action) pairs up front:
    a generation loop that follows finds every pair cached, and its frames and cache contents are bitwise
    those of a context that computes the pairs on demand."""
    from paper_2506_01380_b200.nfd import NFD
    torch = _torch()
    cfg = I.make_cfg(name)
    w = I.make_weights(cfg, 11, "stress")
    warm, cold = NFD(cfg, w), NFD(cfg, w)
    n_pairs = (cfg["n_steps"] + 1) * cfg["n_actions"]
    assert warm.warm_modulation() == n_pairs
    assert warm.warm_modulation() == 0                      # all cached already
    _, m0 = warm.cond_cache_stats()
    fs = I.frame_shape(cfg)
    for step in range(6):
        k = 1 + step % 2
        noise = dev(I.make_latents(cfg, cfg["n_steps"] * k, 40 + step).reshape((cfg["n_steps"], k) + fs))
        cz = dev(I.make_latents(cfg, k, 60 + step))
        a = (3 * step + 1) % cfg["n_actions"]
        ya, yb = warm.speculate(k, a, noise, cz), cold.speculate(k, a, noise, cz)
        assert torch.equal(ya, yb)
        warm.rollback(k), cold.rollback(k)
    assert warm.cond_cache_stats()[1] == m0, "no pair may be missing after the warm-up"
    assert cold.cond_cache_stats()[1] > 0
    assert warm.kv_hash() == cold.kv_hash()
    assert warm.status() == 0 and cold.status() == 0


@pytest.mark.parametrize("name", ["tiny_bf16", "tiny", "nfd310m_slice"])
def test_deferred_commit_equals_immediate_commit(name):
    """A speculation leaves the commit of its frames to the first pass of the next speculation (the paper's
    "compute and cache their KVs during the first denoising step", Appendix on KV caching).  Frames, counters
    and cache contents must be bitwise those of a context that commits at once, whatever mix of k and
    accepted counts is used, and whatever call forces the deferred pages to be written."""
    from paper_2506_01380_b200.nfd import NFD
    torch = _torch()
    cfg = I.make_cfg(name)
    w = I.make_weights(cfg, 7, "stress")
    lazy, eager = NFD(cfg, w), NFD(cfg, w)
    eager.set_option("lazy_commit", 0)
    x0 = dev(I.make_latents(cfg, 2, 11))
    for g in (lazy, eager):
        g.commit_frame(x0, [1, 2], dev(I.make_latents(cfg, 2, 12)))
    S = cfg["n_steps"]
    plan = [(2, 1), (1, 1), (3, 3), (4, 2), (1, 1), (2, 2)]          # (k, accepted)
    for step, (k, n_acc) in enumerate(plan):
        noise = dev(I.make_noise(cfg, S, k, 100 + step))
        cz = dev(I.make_latents(cfg, k, 200 + step)) if step % 2 == 0 else None
        ya = lazy.speculate(k, step % cfg["n_actions"], noise, cz)
        yb = eager.speculate(k, step % cfg["n_actions"], noise, cz)
        assert torch.equal(ya, yb), f"speculation {step}: frames differ"
        assert lazy.kv_state() == eager.kv_state()
        lazy.rollback(n_acc)
        eager.rollback(n_acc)
        assert lazy.kv_state() == eager.kv_state()
        if step == 3:                                                 # forces the deferred pages out mid-way
            assert lazy.kv_hash() == eager.kv_hash()
    assert lazy.kv_hash() == eager.kv_hash()
    L, total = cfg["n_layers"], lazy.kv_state()[0]
    for f in (total - 1, total - 2):
        Ka, Va = lazy.kv_read(L - 1, f)
        Kb, Vb = eager.kv_read(L - 1, f)
        assert torch.equal(Ka, Kb) and torch.equal(Va, Vb)
    assert lazy.status() == 0 and eager.status() == 0


def test_batch8_streams_at_model_width_match_single_streams():
    """Batched decoding (8 independent streams, 32-frame context) on a 2-layer slice of the 310M-class
    width: one batched speculation must give bitwise the frames and caches of eight single-stream ones."""
    from paper_2506_01380_b200.nfd import NFD
    torch = _torch()
    cfg = I.make_cfg("nfd310m_b8", n_layers=2)
    w = I.make_weights(cfg, 9, "stress")
    gb, gs = NFD(cfg, w), NFD(cfg, w)
    S, k, n = cfg["n_steps"], 1, 8
    for s in range(n):
        x0 = dev(I.round_bf16(I.make_latents(cfg, 2, 300 + s)))
        acts = I.make_actions_uniform(cfg, 2, 400 + s)
        gb.commit_frame(x0, acts, None, stream=s)
        gs.commit_frame(x0, acts, None, stream=s)
    noise = dev(I.round_bf16(np.stack([I.make_noise(cfg, S, k, 500 + s) for s in range(n)], axis=1)))   # [S,n,k,...]
    actions = [(3 * s + 1) % cfg["n_actions"] for s in range(n)]
    xb = gb.speculate_batched(list(range(n)), k, actions, noise)
    for s in range(n):
        xs = gs.speculate(k, actions[s], noise[:, s].contiguous(), stream=s)
        assert torch.equal(xs, xb[s]), f"stream {s}"
    for s in range(n):
        gb.rollback(1, stream=s)
        gs.rollback(1, stream=s)
        assert gb.kv_state(s) == gs.kv_state(s) == (3, 0, 0)
        assert gb.kv_hash(s) == gs.kv_hash(s)
    assert gb.status() == 0 and gs.status() == 0
