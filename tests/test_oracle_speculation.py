"""Pins for the oracle's speculation / rollback bookkeeping (CPU only)."""
import itertools

import numpy as np

from oracle import nfd_oracle as O
from paper_2506_01380_b200 import inputs as I


def micro_cfg():
    return I.make_cfg("tiny", n_layers=1, latent_h=2, latent_w=2, d_model=32, n_heads=1, d_mlp=32,
                      ctx_frames=2, max_spec=4, n_actions=2)


def noise_for(cfg, i, k):
    # noise is a function of the absolute frame index so that every run sees the
    # same noise for the same frame, however the frames are grouped into passes
    S = cfg["n_steps"]
    return np.stack([np.concatenate([I.make_noise(cfg, 1, 1, 1000 * (i + j) + s)[0] for j in range(k)])
                     for s in range(S)])


def ctx_noise_for(cfg, i, k):
    return np.concatenate([I.make_latents(cfg, 1, 77000 + i + j) for j in range(k)])


def test_rollback_equals_never_having_speculated():
    cfg = micro_cfg()
    w = I.make_weights(cfg, 0, "stress")
    for n in range(1, 6):
        for acts in itertools.product([0, 1], repeat=n):
            for k in (2, 4):
                a = O.NFDOracle(cfg, w)
                frames, spec, acc, passes = a.generate(list(acts), n, k,
                                                       lambda i, kk: noise_for(cfg, i, kk),
                                                       lambda i, kk: ctx_noise_for(cfg, i, kk))
                assert len(frames) == n == acc and a.n_committed == n and a.n_tentative == 0
                # replay: speculate exactly the accepted prefix each time (no rejected frame is ever computed)
                b = O.NFDOracle(cfg, w)
                i = 0
                ref = []
                while i < n:
                    m = O.accepted_count(list(acts), i, min(k, n - i))
                    x0 = b.speculate(m, acts[i], noise_for(cfg, i, m), ctx_noise_for(cfg, i, m))
                    b.rollback(m)
                    ref.extend(list(x0))
                    i += m
                # (numpy's matmul rounds differently for different batch sizes, so
                # values are compared to 1e-12 rather than through the digest)
                assert (a.n_committed, a.n_tentative) == (b.n_committed, b.n_tentative)
                for l in range(cfg["n_layers"]):
                    assert sorted(f for f in a.kv[l] if f >= a.window_first()) == \
                        sorted(f for f in b.kv[l] if f >= b.window_first())
                    for f in range(a.window_first(), a.n_total):
                        for x, y in zip(a.kv_frame(l, f), b.kv_frame(l, f)):
                            np.testing.assert_allclose(x, y, atol=1e-12)
                for fa, fb in zip(frames, ref):
                    np.testing.assert_allclose(fa, fb, atol=1e-12)


def test_rollback_zero_and_counters():
    cfg = micro_cfg()
    orc = O.NFDOracle(cfg, I.make_weights(cfg, 0, "stress"))
    orc.commit_frame(I.make_latents(cfg, 2, 1).astype(float), [0, 1])
    d0 = orc.kv_digest()
    orc.speculate(3, 1, noise_for(cfg, 2, 3))
    assert (orc.n_committed, orc.n_tentative, orc.window_first()) == (2, 3, 3)
    orc.rollback(0)
    assert (orc.n_committed, orc.n_tentative, orc.window_first()) == (2, 0, 0)
    assert orc.kv_digest() == d0


def test_k1_speculation_is_plain_generation():
    # k = 1: the sampler followed by a commit; compare with the steps written out.
    cfg = micro_cfg()
    w = I.make_weights(cfg, 3, "stress")
    a, b = O.NFDOracle(cfg, w), O.NFDOracle(cfg, w)
    nz = noise_for(cfg, 0, 1).astype(float)
    cz = ctx_noise_for(cfg, 0, 1).astype(float)
    x0 = a.speculate(1, 1, nz, cz)
    a.rollback(1)
    sd = cfg["sigma_d"]
    x = sd * nz[0]
    sched = O.trig_schedule(cfg["n_steps"])
    for s, tp in enumerate(sched):
        t = O.fm_time(tp)
        x_in = O.fm_input(x, tp, sd)
        v = b.denoise_step(x_in, t, 1)
        est = sd * (x_in - t * v)
        if s + 1 < len(sched):
            x = O.renoise(est, nz[s + 1], sched[s + 1], sd)
    np.testing.assert_allclose(x0, est, atol=1e-12)
    b.commit_frame(est, [1], cz)
    for l in range(cfg["n_layers"]):
        np.testing.assert_allclose(a.kv_frame(l, 0)[0], b.kv_frame(l, 0)[0], atol=1e-12)
        np.testing.assert_allclose(a.kv_frame(l, 0)[1], b.kv_frame(l, 0)[1], atol=1e-12)


# ---------------------------------------------------------------- the undistilled sampler's wrapper
def test_dpmpp_wrapper_equals_the_solver_driven_by_hand():
    """NFDOracle.sample_dpmpp (Section 3.2 "Sampling") against a twin oracle on which the steps are taken one
    by one: the model is evaluated on the unit-variance state at the grid's times, the data prediction is
    x - t v, the solver's result is scaled by sigma_d, and the k frames are committed as tentative."""
    cfg = micro_cfg()
    w = I.make_weights(cfg, 5, "stress")
    a, b = O.NFDOracle(cfg, w), O.NFDOracle(cfg, w)
    prompt = I.make_latents(cfg, 2, 9).astype(float)
    for o in (a, b):
        o.commit_frame(prompt, [0, 1], None)
    k, n_evals, act = 2, 6, 1
    nz = np.concatenate([I.make_latents(cfg, 1, 400 + j) for j in range(k)]).astype(float)
    cz = ctx_noise_for(cfg, 2, k).astype(float)
    x0 = a.sample_dpmpp(k, act, nz, n_evals=n_evals, ctx_noise=cz)
    assert (a.n_committed, a.n_tentative) == (2, k)
    # by hand on the twin: every evaluation is a plain denoise_step on top of the two committed frames
    seen = []

    def x0_fn(x, t):
        seen.append(t)
        assert (b.n_committed, b.n_tentative) == (2, 0)
        return x - t * b.denoise_step(x, t, act)

    est = cfg["sigma_d"] * O.dpmpp_2m(x0_fn, nz, n_evals)
    assert seen == O.dpmpp_grid(n_evals)[:-1]
    np.testing.assert_allclose(x0, est, atol=1e-12)
    b.commit_frame(est, [act] * k, cz)            # same pages, counted as committed instead of tentative
    for l in range(cfg["n_layers"]):
        for f in (2, 3):
            np.testing.assert_allclose(a.kv_frame(l, f)[0], b.kv_frame(l, f)[0], atol=1e-12)
            np.testing.assert_allclose(a.kv_frame(l, f)[1], b.kv_frame(l, f)[1], atol=1e-12)
    a.rollback(1)
    assert (a.n_committed, a.n_tentative) == (3, 0) and 3 not in a.kv[0]


def test_dpmpp_wrapper_closed_form_for_a_constant_velocity():
    """With every gate of the blocks and the output matrix set to zero the velocity is the output bias b,
    whatever the input: the probability-flow path is the straight line x(t) = x(1) - (1 - t) b, the data
    prediction x - t v is the constant x(1) - b along it, and a data-prediction solver returns exactly that.
    So the generated frame is sigma_d (noise - b): this fixes the sign of x0 = x - t v, that the start is the
    unit-variance noise itself and that the result is scaled by sigma_d once."""
    cfg = micro_cfg()
    w = I.make_weights(cfg, 6, "stress")
    d = cfg["d_model"]
    for l in range(cfg["n_layers"]):
        w[f"w_mod.{l}"][:, 2 * d:3 * d] = 0.0
        w[f"w_mod.{l}"][:, 5 * d:6 * d] = 0.0
        w[f"b_mod.{l}"][2 * d:3 * d] = 0.0
        w[f"b_mod.{l}"][5 * d:6 * d] = 0.0
    w["w_out"][:] = 0.0
    o = O.NFDOracle(cfg, w)
    nz = I.make_latents(cfg, 1, 31).astype(float)
    # b_out per patch element, laid out as a latent frame (patch = 1 here: one channel vector per token)
    b_frame = o.unpatchify(np.tile(np.asarray(w["b_out"], float), (o.T, 1)))
    for n_evals in (1, 3, 18):
        o.reset()
        x0 = o.sample_dpmpp(1, 0, nz, n_evals=n_evals)
        np.testing.assert_allclose(x0, cfg["sigma_d"] * (nz - b_frame), atol=1e-12)
