"""Pins for the oracle's forward pass (CPU only, fp64, tiny shapes).

The model output has no printed reference in the paper, so the oracle is tied
down by: (1) dense-mask full-sequence forward == incremental cached decoding,
(2) intra-frame permutation equivariance without positional terms, (3) a joint
k-frame pass == k sequential single-frame passes, (4) softmax rows sum to one,
(5) causality, (6) RoPE relativity, (7) special cases equal to a plain pre-LN
transformer written independently below, (8) brute-force loops for the
elementwise and layout pieces."""
import math

import numpy as np
import pytest

from oracle import nfd_oracle as O
from paper_2506_01380_b200 import inputs as I

TOL = 1e-10


def small_cfg(**kw):
    base = dict(latent_h=4, latent_w=4, d_model=64, n_heads=2, d_mlp=96, ctx_frames=3, max_spec=4)
    base.update(kw)
    return I.make_cfg("tiny", **base)


def make(cfg, seed=0, kind="stress", **kw):
    return O.NFDOracle(cfg, I.make_weights(cfg, seed, kind), **kw)


def ctx_inputs(orc, x0, z):
    tp = orc.cfg["t_ctx_trig"]
    return O.fm_input(O.renoise(x0, z, tp, orc.sigma_d), tp, orc.sigma_d), O.fm_time(tp)


# ---------------------------------------------------------------- (1)
@pytest.mark.parametrize("kind,act", [("paper", 0), ("stress", 0), ("stress", 1)])
def test_dense_mask_equals_incremental_cache(kind, act):
    cfg = small_cfg(act=act, d_mlp=96 if act == 0 else 100)
    W = cfg["ctx_frames"]
    n_ctx = W + 4                                  # eviction is exercised
    orc = make(cfg, 1, kind)
    x0 = I.make_latents(cfg, n_ctx, 10).astype(np.float64)
    z = I.make_latents(cfg, n_ctx, 11).astype(np.float64)
    acts = I.make_actions_uniform(cfg, n_ctx + 1, 12)
    # incremental: commit frames in groups of 1, 3, 1, 2 then denoise one new frame
    i = 0
    for n in (1, 3, 1, 2):
        orc.commit_frame(x0[i:i + n], acts[i:i + n], z[i:i + n])
        i += n
    assert i == n_ctx and orc.n_committed == n_ctx and orc.window_first() == n_ctx - W
    x_t = I.make_latents(cfg, 1, 13).astype(np.float64)
    t_new = 0.7
    v_inc = orc.denoise_step(x_t, t_new, int(acts[n_ctx]))
    # dense: all frames in one pass with the explicit mask
    dense = make(cfg, 1, kind)
    x_ctx, t_ctx = ctx_inputs(dense, x0, z)
    X = np.concatenate([x_ctx, x_t])
    v_all, aux = dense.forward_full(X, [t_ctx] * n_ctx + [t_new], list(acts), return_aux=True)
    np.testing.assert_allclose(v_inc[0], v_all[-1], atol=TOL)
    T = orc.T
    for l in range(cfg["n_layers"]):
        for f in range(n_ctx + 1 - W - 1, n_ctx + 1):
            K, V = orc.kv_frame(l, f)
            np.testing.assert_allclose(K, aux["K"][l][:, f * T:(f + 1) * T], atol=TOL)
            np.testing.assert_allclose(V, aux["V"][l][:, f * T:(f + 1) * T], atol=TOL)


def test_window_actually_limits_context():
    # With W small, a far-past frame must not influence the new frame's attention;
    # with a large W it does.  Guards against a mask that ignores W.
    outs = []
    for W in (1, 8):
        cfg = small_cfg(ctx_frames=W, n_layers=1)
        orc = make(cfg, 2)
        X = I.make_latents(cfg, 4, 3).astype(np.float64)
        v1 = orc.forward_full(X, [0.3] * 4, [0, 1, 2, 3])
        X2 = X.copy()
        X2[0] += 1.0
        v2 = orc.forward_full(X2, [0.3] * 4, [0, 1, 2, 3])
        outs.append(np.abs(v1[3] - v2[3]).max())
    assert outs[0] == 0.0 and outs[1] > 1e-6


# ---------------------------------------------------------------- (2)
def test_intra_frame_permutation_equivariance():
    cfg = small_cfg()
    X = I.make_latents(cfg, 3, 5).astype(np.float64)
    t, u = [0.2, 0.2, 0.9], [1, 2, 3]
    T = 16
    perm = np.random.default_rng(0).permutation(T)
    Xp = X.copy()
    g = 1
    Xp[g] = X[g].reshape(4, T)[:, perm].reshape(4, 4, 4)
    for use_rope, should_hold in ((False, True), (True, False)):
        orc = make(cfg, 4, use_rope=use_rope)
        v, vp = orc.forward_full(X, t, u), orc.forward_full(Xp, t, u)
        err_g = np.abs(vp[g].reshape(4, T) - v[g].reshape(4, T)[:, perm]).max()
        err_o = max(np.abs(vp[0] - v[0]).max(), np.abs(vp[2] - v[2]).max())
        if should_hold:
            assert err_g < TOL and err_o < TOL
        else:
            assert err_g > 1e-6                      # positional terms break it: RoPE is doing something


# ---------------------------------------------------------------- (3)
def test_joint_pass_equals_sequential_single_frame_passes():
    cfg = small_cfg()
    orc_a, orc_b = make(cfg, 6), make(cfg, 6)
    x0 = I.make_latents(cfg, 2, 20).astype(np.float64)
    for o in (orc_a, orc_b):
        o.commit_frame(x0, [3, 4])
    k = 3
    x_t = I.make_latents(cfg, k, 21).astype(np.float64)
    v_joint = orc_a.denoise_step(x_t, 0.6, 5)
    for j in range(k):
        v_j = orc_b.denoise_step(x_t[j:j + 1], 0.6, 5, offset=j)
        np.testing.assert_allclose(v_j[0], v_joint[j], atol=TOL)
    for l in range(cfg["n_layers"]):
        for f in range(2, 2 + k):
            np.testing.assert_allclose(orc_a.kv_frame(l, f)[0], orc_b.kv_frame(l, f)[0], atol=TOL)


# ---------------------------------------------------------------- (4)
def test_softmax_rows_and_mask_density():
    cfg = small_cfg(ctx_frames=16)
    orc = make(cfg, 7)
    Fn, T = 6, 16
    X = I.make_latents(cfg, Fn, 8).astype(np.float64)
    _, aux = orc.forward_full(X, [0.5] * Fn, [0] * Fn, return_aux=True)
    fid = np.repeat(np.arange(Fn), T)
    for Pm in aux["P"]:
        assert np.abs(Pm.sum(-1) - 1.0).max() < 1e-14
        masked = fid[None, :] > fid[:, None]
        assert np.all(Pm[:, masked] == 0.0)
        assert np.all(Pm[:, ~masked] > 0.0)
    # block-causal keeps (F+1)/(2F) of the full attention matrix: the "50 %" of Section 3.1
    assert (~masked).mean() == pytest.approx((Fn + 1) / (2 * Fn))


# ---------------------------------------------------------------- (5)
def test_causality():
    cfg = small_cfg(ctx_frames=8)
    orc = make(cfg, 9)
    X = I.make_latents(cfg, 4, 30).astype(np.float64)
    t, u = [0.1, 0.4, 0.6, 0.9], [0, 1, 2, 3]
    v = orc.forward_full(X, t, u)
    X2 = X.copy()
    X2[2] += 0.5
    v2 = orc.forward_full(X2, t, u)
    assert np.abs(v2[:2] - v[:2]).max() == 0.0
    assert np.abs(v2[2] - v[2]).max() > 1e-6 and np.abs(v2[3] - v[3]).max() > 1e-9
    # a later frame's action or time does not reach earlier frames either
    v3 = orc.forward_full(X, [0.1, 0.4, 0.6, 0.2], [0, 1, 2, 7])
    assert np.abs(v3[:3] - v[:3]).max() == 0.0 and np.abs(v3[3] - v[3]).max() > 1e-6


# ---------------------------------------------------------------- (6)
def test_rope_relativity_in_frame_index():
    cfg = small_cfg(ctx_frames=8)
    orc = make(cfg, 10)
    X = I.make_latents(cfg, 3, 31).astype(np.float64)
    a = orc.forward_full(X, [0.3] * 3, [1, 1, 2], frame0=0)
    b = orc.forward_full(X, [0.3] * 3, [1, 1, 2], frame0=41)
    np.testing.assert_allclose(a, b, atol=1e-9)


# ---------------------------------------------------------------- (7) independent plain transformer
def _ref_rope(x, fr, r, c, cfg):
    """Independent formulation: adjacent pairs as complex numbers times e^{i*angle}."""
    H, n, dh = x.shape
    out = np.empty_like(x)
    off = 0
    for n_ax, pos in ((cfg["rope_t"], fr), (cfg["rope_h"], r), (cfg["rope_w"], c)):
        for i in range(n_ax // 2):
            ang = np.asarray(pos, float) * cfg["rope_theta"] ** (-(2 * i) / n_ax)
            zc = (x[:, :, off + 2 * i] + 1j * x[:, :, off + 2 * i + 1]) * np.exp(1j * ang)[None]
            out[:, :, off + 2 * i], out[:, :, off + 2 * i + 1] = zc.real, zc.imag
        off += n_ax
    return out


def _ref_plain_transformer(cfg, w, X, n_layers):
    """Pre-LN transformer, block-causal over frames, no modulation (shift=scale=0, gate=1)."""
    Fn = X.shape[0]
    C, Hh, Ww, p, d, H, dh = cfg["latent_c"], cfg["latent_h"], cfg["latent_w"], cfg["patch"], cfg["d_model"], cfg["n_heads"], cfg["head_dim"]
    th, tw = Hh // p, Ww // p
    T = th * tw
    tok = np.zeros((Fn * T, C * p * p))
    fr, rr, cc = [], [], []
    for f in range(Fn):
        for i in range(th):
            for j in range(tw):
                vec = [X[f, ch, i * p + py, j * p + px] for ch in range(C) for py in range(p) for px in range(p)]
                tok[f * T + i * tw + j] = vec
                fr.append(f), rr.append(i), cc.append(j)
    z = tok @ w["w_pe"] + w["b_pe"]

    def ln(x):
        return (x - x.mean(-1, keepdims=True)) / np.sqrt(x.var(-1, keepdims=True) + cfg["norm_eps"])

    block = np.kron(np.tril(np.ones((Fn, Fn))), np.ones((T, T))) > 0
    for l in range(n_layers):
        qkv = ln(z) @ w[f"w_qkv.{l}"] + w[f"b_qkv.{l}"]
        q, k, v = [qkv[:, i * d:(i + 1) * d].reshape(-1, H, dh).transpose(1, 0, 2) for i in range(3)]
        q, k = _ref_rope(q, fr, rr, cc, cfg), _ref_rope(k, fr, rr, cc, cfg)
        o = np.zeros((Fn * T, d))
        for h in range(H):
            s = q[h] @ k[h].T / math.sqrt(dh)
            s = np.where(block, s, -1e300)
            e = np.exp(s - s.max(-1, keepdims=True))
            o[:, h * dh:(h + 1) * dh] = (e / e.sum(-1, keepdims=True)) @ v[h]
        z = z + o @ w[f"w_o.{l}"] + w[f"b_o.{l}"]
        hmid = ln(z) @ w[f"w_fc1.{l}"] + w[f"b_fc1.{l}"]
        if cfg.get("act", 0) == 0:
            hmid = np.array([[0.5 * a * (1 + math.erf(a / math.sqrt(2))) for a in row] for row in hmid])
        else:       # gated: columns [0, dm) gate, [dm, 2 dm) up; scalar loops on purpose
            dm = cfg["d_mlp"]
            hmid = np.array([[row[i] / (1 + math.exp(-row[i])) * row[dm + i] for i in range(dm)] for row in hmid])
        z = z + hmid @ w[f"w_fc2.{l}"] + w[f"b_fc2.{l}"]
    y = ln(z) @ w["w_out"] + w["b_out"]
    out = np.zeros_like(X)
    for f in range(Fn):
        for i in range(th):
            for j in range(tw):
                vec = y[f * T + i * tw + j].reshape(C, p, p)
                out[f, :, i * p:(i + 1) * p, j * p:(j + 1) * p] = vec
    return out


@pytest.mark.parametrize("patch,act", [(1, 0), (2, 0), (1, 1)])
def test_unmodulated_model_is_a_plain_pre_ln_transformer(patch, act):
    cfg = small_cfg(ctx_frames=8, patch=patch, act=act, d_mlp=96 if act == 0 else 100)
    w = {k: v.astype(np.float64) for k, v in I.make_weights(cfg, 11, "stress").items()}
    d = cfg["d_model"]
    for l in range(cfg["n_layers"]):
        w[f"w_mod.{l}"][:] = 0
        w[f"b_mod.{l}"][:] = 0
        w[f"b_mod.{l}"][2 * d:3 * d] = 1
        w[f"b_mod.{l}"][5 * d:6 * d] = 1
    w["w_fmod"][:] = 0
    w["b_fmod"][:] = 0
    X = I.make_latents(cfg, 3, 32).astype(np.float64)
    got = O.NFDOracle(cfg, w).forward_full(X, [0.2, 0.5, 0.8], [0, 3, 5])
    want = _ref_plain_transformer(cfg, w, X, cfg["n_layers"])
    np.testing.assert_allclose(got, want, atol=1e-9)
    # zero gates: every block is the identity, the output is the final layer of the embedding
    for l in range(cfg["n_layers"]):
        w[f"b_mod.{l}"][:] = 0
    got0 = O.NFDOracle(cfg, w).forward_full(X, [0.2, 0.5, 0.8], [0, 3, 5])
    np.testing.assert_allclose(got0, _ref_plain_transformer(cfg, w, X, 0), atol=1e-9)


def test_modulation_enters_as_scale_shift_gate():
    # One layer, one frame: restate the adaLN-zero block directly.
    cfg = small_cfg(n_layers=1)
    w = {k: v.astype(np.float64) for k, v in I.make_weights(cfg, 12, "stress").items()}
    orc = O.NFDOracle(cfg, w)
    X = I.make_latents(cfg, 1, 33).astype(np.float64)
    t, u = 0.35, 6
    got = orc.forward_full(X, [t], [u])
    d, H, dh = cfg["d_model"], cfg["n_heads"], cfg["head_dim"]
    # conditioning, restated
    i = np.arange(128)
    a = 1000.0 * t * np.exp(-math.log(10000.0) * i / 128)
    emb = np.concatenate([np.cos(a), np.sin(a)])
    sil = lambda x: x * (1 / (1 + np.exp(-x)))
    c = sil(emb @ w["w_t1"] + w["b_t1"]) @ w["w_t2"] + w["b_t2"] + w["a_emb"][u]
    m = sil(c) @ w["w_mod.0"] + w["b_mod.0"]
    sh1, sc1, g1, sh2, sc2, g2 = [m[j * d:(j + 1) * d] for j in range(6)]
    ln = lambda x: (x - x.mean(-1, keepdims=True)) / np.sqrt(x.var(-1, keepdims=True) + 1e-6)
    tok = X[0].reshape(cfg["latent_c"], -1).T          # patch 1: token = channels at a pixel
    z = tok @ w["w_pe"] + w["b_pe"]
    h = ln(z) * (1 + sc1) + sh1
    qkv = h @ w["w_qkv.0"] + w["b_qkv.0"]
    q, k, v = [qkv[:, j * d:(j + 1) * d].reshape(-1, H, dh).transpose(1, 0, 2) for j in range(3)]
    rr, cc = np.divmod(np.arange(16), 4)
    q, k = _ref_rope(q, np.zeros(16), rr, cc, cfg), _ref_rope(k, np.zeros(16), rr, cc, cfg)
    s = q @ k.transpose(0, 2, 1) / math.sqrt(dh)
    e = np.exp(s - s.max(-1, keepdims=True))
    o = ((e / e.sum(-1, keepdims=True)) @ v).transpose(1, 0, 2).reshape(16, d)
    z = z + g1 * (o @ w["w_o.0"] + w["b_o.0"])
    h = ln(z) * (1 + sc2) + sh2
    from scipy.stats import norm as gauss
    hm = h @ w["w_fc1.0"] + w["b_fc1.0"]
    z = z + g2 * ((hm * gauss.cdf(hm)) @ w["w_fc2.0"] + w["b_fc2.0"])   # GELU(x) = x * Phi(x)
    mf = sil(c) @ w["w_fmod"] + w["b_fmod"]
    y = (ln(z) * (1 + mf[d:]) + mf[:d]) @ w["w_out"] + w["b_out"]
    want = y.T.reshape(X.shape)
    np.testing.assert_allclose(got, want, atol=1e-9)


def test_rmsnorm_variant():
    cfg = small_cfg(norm=1)
    orc = make(cfg, 13)
    x = np.random.default_rng(1).standard_normal((5, 64))
    want = x / np.sqrt((x ** 2).sum(-1, keepdims=True) / 64 + 1e-6)
    np.testing.assert_allclose(orc.norm(x), want, atol=1e-14)


# ---------------------------------------------------------------- (8)
def test_standalone_attention_reduces_to_textbook():
    q, k, v = I.make_qkv(2, 16, 7, 7, seed=3, bf16=False)
    got = O.attention_block_causal(q, k, v, np.zeros(7, int), np.zeros(7, int), 4)
    for h in range(2):
        s = q[h].astype(float) @ k[h].astype(float).T / 4.0
        p = np.exp(s) / np.exp(s).sum(-1, keepdims=True)
        np.testing.assert_allclose(got[h], p @ v[h], atol=1e-12)
    # frame-granular mask by brute force
    qf, kf = np.array([2, 2, 3]), np.array([0, 0, 1, 2, 2, 3, 3])
    q, k, v = I.make_qkv(1, 8, 3, 7, seed=4, bf16=False)
    got = O.attention_block_causal(q, k, v, qf, kf, window=1)
    for i in range(3):
        vis = [j for j in range(7) if qf[i] - 1 <= kf[j] <= qf[i]]
        s = np.array([float(q[0, i].astype(float) @ k[0, j].astype(float)) / math.sqrt(8) for j in vis])
        p = np.exp(s - s.max())
        p /= p.sum()
        np.testing.assert_allclose(got[0, i], sum(p[a] * v[0, j].astype(float) for a, j in enumerate(vis)), atol=1e-12)


def test_patchify_roundtrip_and_order():
    cfg = small_cfg(patch=2)
    orc = make(cfg, 14)
    X = I.make_latents(cfg, 2, 40).astype(np.float64)
    tok = orc.patchify(X)
    assert tok.shape == (2 * 4, 4 * 4)
    # token (f=1, row=1, col=0), element (c=2, py=1, px=0)
    assert tok[1 * 4 + 1 * 2 + 0, 2 * 4 + 1 * 2 + 0] == X[1, 2, 1 * 2 + 1, 0 * 2 + 0]
    np.testing.assert_array_equal(orc.unpatchify(tok), X)


def test_gated_mlp_special_cases():
    """The gated feed-forward (act = 1): with the up projection forced to the constant 1 it is a plain SiLU
    MLP; with the gate pre-activation forced to a large constant it is linear in the up projection
    (SiLU(c) -> c); shapes are [d, 2 dm] with the gate columns first."""
    rng = np.random.default_rng(3)
    d, dm, n = 12, 10, 7
    h = rng.standard_normal((n, d))
    w1, b1 = rng.standard_normal((d, 2 * dm)), rng.standard_normal(2 * dm)
    w2, b2 = rng.standard_normal((dm, d)), rng.standard_normal(d)
    # general case against scalar loops
    want = np.zeros((n, d))
    for r in range(n):
        a = [sum(h[r, k] * w1[k, c] for k in range(d)) + b1[c] for c in range(2 * dm)]
        g = [a[i] / (1 + math.exp(-a[i])) * a[dm + i] for i in range(dm)]
        want[r] = [sum(g[i] * w2[i, o] for i in range(dm)) + b2[o] for o in range(d)]
    np.testing.assert_allclose(O.mlp(h, w1, b1, w2, b2, 1), want, atol=1e-12)
    # up == 1: plain SiLU MLP
    w1u, b1u = w1.copy(), b1.copy()
    w1u[:, dm:], b1u[dm:] = 0.0, 1.0
    a = h @ w1[:, :dm] + b1[:dm]
    np.testing.assert_allclose(O.mlp(h, w1u, b1u, w2, b2, 1), (a / (1 + np.exp(-a))) @ w2 + b2, atol=1e-12)
    # gate pre-activation == 40: SiLU(40) = 40 to 1e-16, so the block is 40 * (h Wu + bu) W2 + b2
    w1g, b1g = w1.copy(), b1.copy()
    w1g[:, :dm], b1g[:dm] = 0.0, 40.0
    np.testing.assert_allclose(O.mlp(h, w1g, b1g, w2, b2, 1), 40.0 * (h @ w1[:, dm:] + b1[dm:]) @ w2 + b2, rtol=1e-12)
    # act 0 is untouched by the new branch
    a0 = h @ w1[:, :dm] + b1[:dm]
    np.testing.assert_allclose(O.mlp(h, w1[:, :dm], b1[:dm], w2, b2, 0), O.gelu(a0) @ w2 + b2, atol=1e-15)


def test_gelu_and_round_bf16():
    x = np.linspace(-6, 6, 101)
    want = np.array([0.5 * a * (1 + math.erf(a / math.sqrt(2))) for a in x])
    np.testing.assert_allclose(O.gelu(x), want, atol=1e-15)
    a = np.array([1.0, 1.00390625, 1.01171875, -3.14159, 1e-20, 65504.0], np.float32)
    r = I.round_bf16(a)
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == np.float32(1.015625)   # ties to even
    assert np.all((r.view(np.uint32) & 0xFFFF) == 0)
    assert np.abs(r - a).max() <= np.abs(a).max() * 2 ** -8
