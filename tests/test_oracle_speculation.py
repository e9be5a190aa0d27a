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
