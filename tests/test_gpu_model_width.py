"""GPU parity at the 310M-class width (d = 1024, 16 heads x 64, 336 tokens per frame) for the
workloads that the small cases do not reach: four frames decoded together (Section 4.2; the
paper's Table 2 goes up to N = 4), batched streams behind a full 32-frame context (Section 5,
"Dataset and Preprocessing"), free-running generation after a 16-frame prompt (Section 4.1
"Sampling" with the control flow of the appendix listing), every kernel of a block against the
oracle's intermediate values, and a residual stream with a large common offset (the folded
LayerNorm's weak spot).  Tolerances are those of tests/test_gpu_parity.py."""
import math

import numpy as np
import pytest

from oracle import nfd_oracle as O
from paper_2506_01380_b200 import inputs as I
from test_gpu_parity import check, dev, make_pair, prompt

pytestmark = pytest.mark.gpu
BF16 = I.DTYPE_BF16


def _kv_check(g, orc, layers, frames, what, stream=0, scale=False):
    worst = 0.0
    for l in layers:
        for f in frames:
            K, V = g.kv_read(l, f, stream=stream)
            a, _ = check(K, orc.kv_frame(l, f)[0], BF16, f"{what} K l{l} f{f}", scale_by_magnitude=scale)
            b, _ = check(V, orc.kv_frame(l, f)[1], BF16, f"{what} V l{l} f{f}", scale_by_magnitude=scale)
            worst = max(worst, a, b)
    return worst


def test_four_frame_pass_and_speculation_at_model_width():
    """Four speculative frames in one pass: k = 4 frames (1344 query rows, block-causal among themselves) on a two-layer slice with
    the stress weights.  First one teacher-forced pass (velocity and the K/V pages it leaves), then a full
    speculation of four frames with two of them accepted, against the oracle doing the same."""
    cfg = I.make_cfg("nfd310m_slice")
    g, orc = make_pair(cfg, 31, "stress")
    prompt(cfg, g, orc, 6, seed=720, group=3)
    L = cfg["n_layers"]
    x_t = I.round_bf16(I.make_latents(cfg, 4, 730))
    t = float(np.float32(O.fm_time(math.pi / 4)))
    v = g.denoise_step(dev(x_t), t, 7)
    check(v, orc.denoise_step(x_t.astype(np.float64), t, 7), BF16, "velocity of the 4-frame pass")
    _kv_check(g, orc, (0, L - 1), (0, 5, 6, 7, 8, 9), "4-frame pass")
    S = cfg["n_steps"]
    noise = I.round_bf16(I.make_noise(cfg, S, 4, 740))
    cz = I.round_bf16(I.make_latents(cfg, 4, 741))
    x0 = g.speculate(4, 9, dev(noise), dev(cz))
    x0_ref = orc.speculate(4, 9, noise.astype(np.float64), cz.astype(np.float64))
    check(x0, x0_ref, BF16, "x0 of speculate(k=4)")
    assert g.kv_state() == (6, 4, 0) == (orc.n_committed, orc.n_tentative, orc.window_first())
    g.rollback(2), orc.rollback(2)
    assert g.kv_state() == (8, 0, 0) == (orc.n_committed, orc.n_tentative, orc.window_first())
    # pages of the two accepted frames: functions of frames the device generated itself (see check())
    worst = _kv_check(g, orc, (0, L - 1), (6, 7), "accepted frames", scale=True)
    print(f"max-abs error of the accepted frames' K/V pages: {worst:.3e}")
    # a second speculation rides on the deferred commit of the accepted frames (a 2 + 3 frame first pass)
    noise = I.round_bf16(I.make_noise(cfg, S, 3, 750))
    x0 = g.speculate(3, 2, dev(noise))
    check(x0, orc.speculate(3, 2, noise.astype(np.float64)), BF16, "x0 of the following speculate(k=3)")
    assert g.status() == 0


def test_batched_streams_behind_a_full_32_frame_context():
    """Batched streams on a two-layer slice: a context made for 8 streams with a 32-frame window.  Three
    of the streams get 34, 37 and 42 committed frames (window full, oldest frames evicted, the last one past
    the ring's wrap-around), then one batched speculation; each stream against an oracle of its own."""
    from paper_2506_01380_b200.nfd import NFD
    cfg = I.make_cfg("nfd310m_b8", n_layers=2)
    w = I.make_weights(cfg, 41, "stress")
    g = NFD(cfg, w)
    streams, counts = [0, 3, 7], [34, 37, 42]
    orcs = [O.NFDOracle(cfg, w) for _ in streams]
    for s, n, orc in zip(streams, counts, orcs):
        x0 = I.round_bf16(I.make_latents(cfg, n, 800 + s))
        z = I.round_bf16(I.make_latents(cfg, n, 810 + s))
        acts = I.make_actions_uniform(cfg, n, 820 + s)
        for i in range(0, n, 4):
            m = min(4, n - i)
            g.commit_frame(dev(x0[i:i + m]), acts[i:i + m], dev(z[i:i + m]), stream=s)
            orc.commit_frame(x0[i:i + m].astype(np.float64), acts[i:i + m], z[i:i + m].astype(np.float64))
        assert g.kv_state(s) == (n, 0, n - 32) == (orc.n_committed, orc.n_tentative, orc.window_first())
    S, k = cfg["n_steps"], 1
    noise = I.round_bf16(np.stack([I.make_noise(cfg, S, k, 830 + s) for s in streams], axis=1))    # [S,n,k,...]
    cz = I.round_bf16(np.stack([I.make_latents(cfg, k, 840 + s) for s in streams]))
    actions = [5, 17, 30]
    x0 = g.speculate_batched(streams, k, actions, dev(noise), dev(cz))
    for i, (s, orc) in enumerate(zip(streams, orcs)):
        ref = orc.speculate(k, actions[i], noise[:, i].astype(np.float64), cz[i].astype(np.float64))
        check(x0[i], ref, BF16, f"x0 of stream {s}")
        g.rollback(1, stream=s), orc.rollback(1)
        n = counts[i]
        assert g.kv_state(s) == (n + 1, 0, n + 1 - 32) == (orc.n_committed, orc.n_tentative, orc.window_first())
        _kv_check(g, orc, (0, 1), (n - 31, n - 1), f"stream {s} context", stream=s)
        _kv_check(g, orc, (0, 1), (n,), f"stream {s} new frame", stream=s, scale=True)
    assert g.status() == 0


def _free_running(cfg, kind, seed, n_prompt, n_gen):
    g, orc = make_pair(cfg, seed, kind)
    g.warm_modulation()
    prompt(cfg, g, orc, n_prompt, seed=900 + seed, group=4)
    S = cfg["n_steps"]
    acts = I.make_actions_uniform(cfg, n_gen, 950 + seed)
    worst = (0.0, 0.0)
    for i in range(n_gen):
        noise = I.round_bf16(I.make_noise(cfg, S, 1, 1000 * seed + i))
        cz = I.round_bf16(I.make_latents(cfg, 1, 2000 * seed + i))
        x0 = g.speculate(1, acts[i], dev(noise), dev(cz))
        ref = orc.speculate(1, acts[i], noise.astype(np.float64), cz.astype(np.float64))
        a, r = check(x0, ref, cfg["dtype"], f"generated frame {i}")
        worst = (max(worst[0], a), max(worst[1], r))
        g.rollback(1), orc.rollback(1)
        assert g.kv_state() == (orc.n_committed, orc.n_tentative, orc.window_first())
    assert g.status() == 0
    print(f"free-running {kind} L={cfg['n_layers']}: worst max-abs {worst[0]:.3e}, worst rel-L2 {worst[1]:.3e}")


def test_free_running_six_layers_stress_weights():
    """16 prompt frames, then 4 frames generated one after the other (each through the 4-step sampler, each
    committed with context noise and seen by the next), six layers at model width, stress weights."""
    _free_running(I.make_cfg("nfd310m", n_layers=6), "stress", seed=3, n_prompt=16, n_gen=4)


def test_free_running_full_depth():
    """The same on all 24 layers of the 310M-class model, with N(0, 0.02^2) weights."""
    _free_running(I.make_cfg("nfd310m"), "paper", seed=4, n_prompt=16, n_gen=4)


@pytest.mark.parametrize("fuse_ln", [1, 0])
def test_every_kernel_of_a_block_against_the_oracle(fuse_ln):
    """One layer at model width, stress weights (every operand of order one), two frames on top of three cached
    ones: each activation buffer that a kernel of the block leaves is compared with the oracle's value of the
    same quantity -- rotated queries (QKV projection + 3D RoPE), K/V pages, attention output, the first MLP
    projection's activation (adaLN folded into that GEMM, or as a kernel of its own), the residual stream
    after the block, and the output of the final adaLN kernel."""
    cfg = I.make_cfg("nfd310m", n_layers=1)
    g, orc = make_pair(cfg, 51, "stress", fuse_ln=fuse_ln)
    prompt(cfg, g, orc, 3, seed=770, group=3)
    k, T, d, H, dh, dm = 2, 336, 1024, 16, 64, 4096
    x_t = I.round_bf16(I.make_latents(cfg, k, 771))
    t, act = 0.4375, 11
    v = g.denoise_step(dev(x_t), t, act)
    v_ref = orc.denoise_step(x_t.astype(np.float64), t, act)
    check(v, v_ref, BF16, "velocity")
    # the oracle's intermediates, from its own building blocks in the order of its forward pass
    w = orc.w
    cvec = np.stack([orc.cond_vector(t, act)] * k)
    sh1, sc1, g1, sh2, sc2, g2 = orc._mod("w_mod.0", "b_mod.0", cvec, 6)
    z0 = orc.patchify(x_t.astype(np.float64)) @ w["w_pe"] + w["b_pe"]
    h1 = orc.norm(z0) * (1.0 + sc1) + sh1
    qkv = h1 @ w["w_qkv.0"] + w["b_qkv.0"]
    fr, r, c = orc.token_pos([3, 4])
    q = orc.rope(orc._heads(qkv[:, :d]), fr, r, c)                              # [H, k*T, dh]
    kf = np.repeat(np.arange(5), T)
    Kc = np.concatenate([orc.kv_frame(0, f)[0] for f in range(5)], axis=1)
    Vc = np.concatenate([orc.kv_frame(0, f)[1] for f in range(5)], axis=1)
    o = O.attention_block_causal(q, Kc, Vc, np.repeat([3, 4], T), kf, cfg["ctx_frames"])
    o = o.transpose(1, 0, 2).reshape(k * T, d)
    z1 = z0 + g1 * (o @ w["w_o.0"] + w["b_o.0"])
    h2 = orc.norm(z1) * (1.0 + sc2) + sh2
    hid = O.gelu(h2 @ w["w_fc1.0"] + w["b_fc1.0"])
    z2 = z1 + g2 * (hid @ w["w_fc2.0"] + w["b_fc2.0"])
    n = k * T
    check(g.debug_read("qbuf", n * d).view(H, n, dh), q, BF16, "rotated queries", scale_by_magnitude=True)
    _kv_check(g, orc, (0,), (3, 4), "pages of the pass", scale=True)
    check(g.debug_read("abuf", n * d).view(n, d), o, BF16, "attention output")
    check(g.debug_read("mbuf", n * dm).view(n, dm), hid, BF16, "MLP activation", scale_by_magnitude=True)
    check(g.debug_read("z", n * d).view(n, d), z2, BF16, "residual stream", scale_by_magnitude=True)
    shf, scf = orc._mod("w_fmod", "b_fmod", cvec, 2)
    check(g.debug_read("hbuf", n * d).view(n, d), orc.norm(z2) * (1.0 + scf) + shf, BF16, "final adaLN",
          scale_by_magnitude=True)
    assert g.status() == 0


@pytest.mark.parametrize("ratio,fuse_ln", [(3.0, 1), (3.0, 0), (30.0, 0)])
def test_residual_stream_with_a_common_offset(ratio, fuse_ln):
    """Every token's residual row gets a common offset of `ratio` standard deviations (through the patch
    embedding's bias).  The folded LayerNorm rounds z (1 + scale) to bf16 before the mean is removed, so its
    error grows with |mean| / std; it is inside the tolerance up to a ratio of a few, which is the range the
    fold is meant for, and the stand-alone LayerNorm (fuse_ln = 0) is the path for anything beyond."""
    cfg = I.make_cfg("nfd310m_slice")
    w = I.make_weights(cfg, 61, "stress")
    # z = patch-embedding of an N(0,1) latent has unit variance per element under these weights
    w["b_pe"] = I.round_bf16(w["b_pe"] + np.float32(ratio))
    from paper_2506_01380_b200.nfd import NFD
    g, orc = NFD(cfg, w), O.NFDOracle(cfg, w)
    g.set_option("fuse_ln", fuse_ln)
    prompt(cfg, g, orc, 3, seed=780, group=3)
    x_t = I.round_bf16(I.make_latents(cfg, 1, 781))
    v = g.denoise_step(dev(x_t), 0.6, 4)
    a, r = check(v, orc.denoise_step(x_t.astype(np.float64), 0.6, 4), BF16, f"velocity at offset {ratio}")
    print(f"offset {ratio} std, fuse_ln {fuse_ln}: max-abs {a:.3e}, rel-L2 {r:.3e}")
    _kv_check(g, orc, (0, 1), (2, 3), f"pages at offset {ratio}", scale=True)
    assert g.status() == 0
