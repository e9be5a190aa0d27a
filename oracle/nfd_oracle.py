"""fp64 CPU oracle for the block-causal diffusion-transformer forward pass.

TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, numpy-fp64 restatement
of what the hot path computes, written from the paper.  It is imported only by
the tests, by the smoke check and by the benchmark's CPU-baseline leg; the
CUDA library never calls it and shares no code with it.

What follows the paper, and where:
  * block-wise causal attention (Section 3.1, "Block-wise Causal Attention"):
    a token attends to every token of its own frame and of earlier frames;
    here additionally limited to the last W earlier frames (the paper evaluates
    with a fixed-length context, Section 5 "Dataset and Preprocessing").
  * adaLN-zero conditioning on timestep + action (Section 3.1, "Action
    Conditioning"), DiT block internals by the DiT citation.
  * 3D rotary embedding (Section 3.1, "3D Positional Embedding"): the head
    dimension is split [n_T, n_H, n_W]; per-axis rotary frequencies are
    concatenated along the last dimension.
  * Flow-Matching <-> TrigFlow conversion (Section 4.1, Eq. for F_theta, the
    unnumbered display defining x^t and t from t', and Eq. "para scm" for
    f_theta), Section 3.2 "Sampling" for the velocity -> clean-frame formula.
  * 4-step sampling (Section 4.1, "Sampling"), speculative sampling
    (Section 4.2 and the appendix listing's control flow), context-noise
    injection (Section 4.3), KV caching of noisy context frames (Appendix,
    "Accelerating Inference via KV Caching").

Parity status: the model output itself is "parity unpinned" against the paper
(the paper prints no weights and no tensors).  It is pinned by the structural
tests in tests/test_oracle_*.py: dense-mask full-sequence forward == incremental
cached decoding, permutation equivariance, joint k-frame pass == k sequential
passes, softmax rows sum to one, causality, RoPE relativity, special cases that
reduce to independently written textbook formulas, and the sampler identities.
"""
from __future__ import annotations

import math
import struct
import zlib

import numpy as np
from scipy.special import erf as _erf

F64 = np.float64


# --------------------------------------------------------------------------
# Sampler algebra (Section 3.2 "Sampling"; Section 4.1)
# --------------------------------------------------------------------------

def fm_time(tp: float) -> float:
    """Flow-Matching time t from TrigFlow time t' (Section 4.1, display after
    the F_theta equation): t = sin t' / (sin t' + cos t')."""
    s, c = math.sin(tp), math.cos(tp)
    return s / (s + c)


def fm_input(x_trig, tp: float, sigma_d: float):
    """Model input x^t from the TrigFlow sample x^{t'} (same display):
    x^t = x^{t'}/sigma_d * sqrt(t^2 + (1-t)^2)."""
    t = fm_time(tp)
    return np.asarray(x_trig, F64) / sigma_d * math.sqrt(t * t + (1.0 - t) * (1.0 - t))


def F_theta(x_t, v, t: float):
    """TrigFlow network output from the velocity (Section 4.1, first equation):
    F = [ (1-2t) x^t + (1-2t+2t^2) v ] / sqrt(t^2+(1-t)^2)."""
    x_t, v = np.asarray(x_t, F64), np.asarray(v, F64)
    return ((1.0 - 2.0 * t) * x_t + (1.0 - 2.0 * t + 2.0 * t * t) * v) / math.sqrt(t * t + (1.0 - t) * (1.0 - t))


def f_theta(x_trig, F, tp: float, sigma_d: float):
    """Clean-data prediction (Section 4.1, Eq. "para scm"):
    f = cos t' * x^{t'} - sin t' * sigma_d * F."""
    return math.cos(tp) * np.asarray(x_trig, F64) - math.sin(tp) * sigma_d * np.asarray(F, F64)


def x0_from_velocity(x_t, v, t: float):
    """Section 3.2 "Sampling": x0 = (x^t - t*eps)/(1-t), eps = (1-t) v + x^t.
    Only defined for t < 1."""
    x_t, v = np.asarray(x_t, F64), np.asarray(v, F64)
    eps = (1.0 - t) * v + x_t
    return (x_t - t * eps) / (1.0 - t)


def trig_schedule(n_steps: int):
    """Section 4.1 "Sampling": timesteps chosen linearly between t'_max = pi/2
    and t'_min = 0.  The sample starts at pi/2; the final denoise lands on 0, so
    the model is evaluated at pi/2 * (S - s)/S, s = 0..S-1."""
    return [0.5 * math.pi * (n_steps - s) / n_steps for s in range(n_steps)]


def renoise(x0, z, tp_next: float, sigma_d: float):
    """Consistency-model multistep sampling (Section 4.1 "Sampling"): after a
    denoise, inject noise for the next timestep.  TrigFlow's forward process is
    x^{t'} = cos t' * x0 + sin t' * sigma_d * z."""
    return math.cos(tp_next) * np.asarray(x0, F64) + math.sin(tp_next) * sigma_d * np.asarray(z, F64)


def dpmpp_grid(n_evals: int):
    """Time grid of the multistep ODE sampler below: t_0 = 1 (pure noise) down to t_M = 0 in M = n_evals equal
    steps of Flow-Matching time; the model is evaluated at t_0 .. t_{M-1}.  (Section 3.2 "Sampling" names the
    solver and, in the experiments, 18 function evaluations; it gives no grid, so equal steps are a reading.)"""
    return [1.0 - i / n_evals for i in range(n_evals + 1)]


def dpmpp_coeffs(t_prev2, t_prev: float, t: float, last: bool):
    """Coefficients (a, b, c) of one step t_prev -> t of DPM-Solver++(2M) (Lu et al. 2022, the multistep
    second-order solver for data-prediction models), written for the Flow-Matching path alpha_t = 1 - t,
    sigma_t = t, lambda_t = ln(alpha_t / sigma_t):
        x_t = (sigma_t / sigma_prev) x_prev - alpha_t (exp(-h) - 1) D,   h = lambda_t - lambda_prev,
        D   = (1 + 1/(2r)) x0(t_prev) - 1/(2r) x0(t_prev2),              r = h_prev / h,
    returned as x_t = a x_prev + b ((1 + c) x0(t_prev) - c x0(t_prev2)).  Where a lambda is infinite (t = 1 at the
    start, t = 0 at the end) the limits are taken: exp(-h) -> 0, and the step is first order (c = 0) when there is
    no finite previous step, which is the first two steps; the last step is first order as well (the customary
    "lower order final" rule; with t = 0 it returns the last data prediction itself)."""
    a = t / t_prev
    # -alpha_t (exp(-h) - 1) with exp(-h) = (alpha_prev / sigma_prev) (sigma_t / alpha_t)
    b = (1.0 - t) - (1.0 - t_prev) * t / t_prev
    c = 0.0
    if t_prev2 is not None and not last and t_prev2 < 1.0 and t > 0.0:
        lam = lambda u: math.log((1.0 - u) / u)
        h, h_prev = lam(t) - lam(t_prev), lam(t_prev) - lam(t_prev2)
        c = h / (2.0 * h_prev)              # 1 / (2 r)
    return a, b, c


def dpmpp_2m(x0_fn, x_T, n_evals: int):
    """DPM-Solver++(2M) over dpmpp_grid from x_T (at t = 1) to t = 0 for a data-prediction function
    x0_fn(x, t).  Returns the sample at t = 0."""
    ts = dpmpp_grid(n_evals)
    x = np.asarray(x_T, F64)
    x0_prev = None
    for i in range(1, n_evals + 1):
        x0_cur = x0_fn(x, ts[i - 1])
        a, b, c = dpmpp_coeffs(ts[i - 2] if i >= 2 else None, ts[i - 1], ts[i], last=(i == n_evals))
        D = (1.0 + c) * x0_cur - (c * x0_prev if c != 0.0 else 0.0)
        x = a * x + b * D
        x0_prev = x0_cur
    return x


def accepted_count(true_actions, i: int, k: int) -> int:
    """Section 4.2 / appendix listing: frames i..i+k-1 were generated under
    action true_actions[i] repeated.  The leading frames whose true action
    equals that action are verified; the first mismatch and everything after it
    are discarded.  Frame i itself always used its true action, so the count is
    at least 1.  Capped by the number of actions available."""
    n = 1
    while n < k and i + n < len(true_actions) and true_actions[i + n] == true_actions[i]:
        n += 1
    return n


# --------------------------------------------------------------------------
# Elementwise pieces
# --------------------------------------------------------------------------

def silu(x):
    return x / (1.0 + np.exp(-x))


def gelu(x):
    """Exact (erf) GELU."""
    return 0.5 * x * (1.0 + _erf(x / math.sqrt(2.0)))


def mlp(h, w1, b1, w2, b2, act: int):
    """Feed-forward of a block.  act 0: GELU(h W1 + b1) W2 + b2.  act 1: the gated form
    (SiLU(h Wg + bg) * (h Wu + bu)) W2 + b2, with W1 = [Wg | Wu] side by side; the paper's size table lists an
    MLP width of about 8/3 of the hidden width for two of its three models, the customary width of this
    form, and names no activation, so the gated form is offered as a reading, not claimed."""
    a = h @ w1 + b1
    if act == 0:
        return gelu(a) @ w2 + b2
    dm = w2.shape[0]
    return (silu(a[:, :dm]) * a[:, dm:]) @ w2 + b2


def softmax_rows(s):
    m = np.max(s, axis=-1, keepdims=True)
    e = np.exp(s - m)
    return e / np.sum(e, axis=-1, keepdims=True)


class NFDOracle:
    """fp64 model + frame cache.  `weights` maps the names of
    `inputs.weight_shapes` to arrays (promoted to fp64 here)."""

    def __init__(self, cfg: dict, weights: dict, use_rope: bool = True):
        self.cfg = dict(cfg)
        self.w = {k: np.asarray(v, F64) for k, v in weights.items()}
        c = cfg
        self.L, self.d, self.H, self.dh = c["n_layers"], c["d_model"], c["n_heads"], c["head_dim"]
        assert self.H * self.dh == self.d
        self.p = c["patch"]
        self.C, self.Hl, self.Wl = c["latent_c"], c["latent_h"], c["latent_w"]
        self.th, self.tw = self.Hl // self.p, self.Wl // self.p
        self.T = self.th * self.tw
        self.P = self.C * self.p * self.p
        self.W = c["ctx_frames"]
        self.kmax = c["max_spec"]
        self.sigma_d = float(c["sigma_d"])
        self.use_rope = use_rope
        assert c["rope_t"] + c["rope_h"] + c["rope_w"] == self.dh
        self.reset()

    # ---------------- cache state ----------------
    def reset(self):
        # kv[l][frame] = (K[H,T,dh], V[H,T,dh]); K is stored rotated.
        self.kv = [dict() for _ in range(self.L)]
        self.n_committed = 0
        self.n_tentative = 0

    @property
    def n_total(self):
        return self.n_committed + self.n_tentative

    def window_first(self):
        return max(0, self.n_total - self.W)

    # ---------------- building blocks ----------------
    def patchify(self, X):
        """[k,C,H,W] -> [k*T, P]; tokens row-major over (row, col); the patch
        vector is ordered (channel, py, px)."""
        k = X.shape[0]
        p = self.p
        x = np.asarray(X, F64).reshape(k, self.C, self.th, p, self.tw, p)
        x = x.transpose(0, 2, 4, 1, 3, 5)
        return x.reshape(k * self.T, self.P)

    def unpatchify(self, Y):
        k = Y.shape[0] // self.T
        p = self.p
        y = Y.reshape(k, self.th, self.tw, self.C, p, p).transpose(0, 3, 1, 4, 2, 5)
        return y.reshape(k, self.C, self.Hl, self.Wl)

    def timestep_embedding(self, t: float):
        half = 128
        i = np.arange(half, dtype=F64)
        freqs = np.exp(-math.log(10000.0) * i / half)
        a = self.cfg["t_scale"] * t * freqs
        return np.concatenate([np.cos(a), np.sin(a)])

    def cond_vector(self, t: float, u: int):
        """Conditioning vector of one frame: timestep embedding MLP plus the
        action embedding (a linear layer applied to a one-hot action)."""
        w = self.w
        e = self.timestep_embedding(t)
        h = silu(e @ w["w_t1"] + w["b_t1"])
        return h @ w["w_t2"] + w["b_t2"] + w["a_emb"][int(u)]

    def norm(self, x):
        eps = self.cfg["norm_eps"]
        if self.cfg["norm"] == 0:
            mu = x.mean(axis=-1, keepdims=True)
            var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
            return (x - mu) / np.sqrt(var + eps)
        ms = (x * x).mean(axis=-1, keepdims=True)
        return x / np.sqrt(ms + eps)

    def rope_angles(self, frames, rows, cols):
        """[n, dh/2] rotation angles: the first rope_t/2 pairs rotate with the
        frame index, the next rope_h/2 with the token row, the last rope_w/2
        with the token column."""
        parts = []
        for n_ax, pos in ((self.cfg["rope_t"], frames), (self.cfg["rope_h"], rows), (self.cfg["rope_w"], cols)):
            i = np.arange(n_ax // 2, dtype=F64)
            freq = self.cfg["rope_theta"] ** (-2.0 * i / n_ax)
            parts.append(np.asarray(pos, F64)[:, None] * freq[None, :])
        return np.concatenate(parts, axis=1)

    def rope(self, x, frames, rows, cols):
        """Rotate adjacent pairs (2i, 2i+1) of x[H, n, dh]."""
        if not self.use_rope:
            return x
        ang = self.rope_angles(frames, rows, cols)
        c, s = np.cos(ang)[None], np.sin(ang)[None]
        xe, xo = x[..., 0::2], x[..., 1::2]
        out = np.empty_like(x)
        out[..., 0::2] = xe * c - xo * s
        out[..., 1::2] = xe * s + xo * c
        return out

    def token_pos(self, frame_ids):
        """Per-token (frame, row, col) for a list of frame indices."""
        k = len(frame_ids)
        fr = np.repeat(np.asarray(frame_ids, F64), self.T)
        r = np.tile(np.repeat(np.arange(self.th), self.tw), k)
        c = np.tile(np.tile(np.arange(self.tw), self.th), k)
        return fr, r, c

    def _mod(self, name_w, name_b, cvecs, n_chunks):
        """adaLN modulation per frame: W * SiLU(c) + b, split into chunks and
        broadcast to that frame's T tokens."""
        m = silu(cvecs) @ self.w[name_w] + self.w[name_b]          # [k, n_chunks*d]
        m = np.repeat(m, self.T, axis=0)                             # [k*T, ...]
        return [m[:, i * self.d:(i + 1) * self.d] for i in range(n_chunks)]

    def _heads(self, y):
        n = y.shape[0]
        return y.reshape(n, self.H, self.dh).transpose(1, 0, 2)      # [H, n, dh]

    def _final(self, z, cvecs):
        sh, sc = self._mod("w_fmod", "b_fmod", cvecs, 2)
        y = (self.norm(z) * (1.0 + sc) + sh) @ self.w["w_out"] + self.w["b_out"]
        return self.unpatchify(y)

    # ---------------- dense, full-sequence definition ----------------
    def forward_full(self, X, t, u, frame0: int = 0, return_aux: bool = False):
        """All F frames at once with an explicit dense banded block-causal mask.

        X [F,C,H,W] model inputs (already FM-scaled), t[F] FM times, u[F]
        actions; frame f has absolute index frame0+f.  Returns v[F,C,H,W]; with
        return_aux also per-layer rotated K, V ([H, F*T, dh]) and the softmax
        probabilities of every layer."""
        Fn = X.shape[0]
        T = self.T
        frames = [frame0 + f for f in range(Fn)]
        cvecs = np.stack([self.cond_vector(t[f], u[f]) for f in range(Fn)])
        z = self.patchify(X) @ self.w["w_pe"] + self.w["b_pe"]
        fr, r, c = self.token_pos(frames)
        fid = np.repeat(np.arange(Fn), T)
        allowed = (fid[None, :] <= fid[:, None]) & (fid[None, :] >= fid[:, None] - self.W)
        M = np.where(allowed, 0.0, -np.inf)
        aux = {"K": [], "V": [], "P": []}
        for l in range(self.L):
            sh1, sc1, g1, sh2, sc2, g2 = self._mod(f"w_mod.{l}", f"b_mod.{l}", cvecs, 6)
            h = self.norm(z) * (1.0 + sc1) + sh1
            qkv = h @ self.w[f"w_qkv.{l}"] + self.w[f"b_qkv.{l}"]
            q = self.rope(self._heads(qkv[:, :self.d]), fr, r, c)
            k = self.rope(self._heads(qkv[:, self.d:2 * self.d]), fr, r, c)
            v = self._heads(qkv[:, 2 * self.d:])
            S = q @ k.transpose(0, 2, 1) / math.sqrt(self.dh) + M[None]
            Pm = softmax_rows(S)
            o = (Pm @ v).transpose(1, 0, 2).reshape(Fn * T, self.d)
            z = z + g1 * (o @ self.w[f"w_o.{l}"] + self.w[f"b_o.{l}"])
            h = self.norm(z) * (1.0 + sc2) + sh2
            m = mlp(h, self.w[f"w_fc1.{l}"], self.w[f"b_fc1.{l}"], self.w[f"w_fc2.{l}"], self.w[f"b_fc2.{l}"],
                    self.cfg.get("act", 0))
            z = z + g2 * m
            if return_aux:
                aux["K"].append(k)
                aux["V"].append(v)
                aux["P"].append(Pm)
        out = self._final(z, cvecs)
        return (out, aux) if return_aux else out

    # ---------------- incremental (cached) form ----------------
    def forward_chunk(self, X, t, u, base: int, store: bool = True, kv_only_last: bool = False):
        """k new frames with absolute indices base..base+k-1 on top of the
        cache.  Frame base+j attends to cached frames in [base+j-W, base-1]
        and to chunk frames 0..j.  The chunk's K/V are written to the cache
        (any older entry for those frame indices is replaced).
        Returns (v[k,C,H,W], newK[l][H,k*T,dh], newV[l])."""
        k = X.shape[0]
        T = self.T
        frames = [base + j for j in range(k)]
        cvecs = np.stack([self.cond_vector(t[j], u[j]) for j in range(k)])
        z = self.patchify(X) @ self.w["w_pe"] + self.w["b_pe"]
        fr, r, c = self.token_pos(frames)
        newK, newV = [], []
        for l in range(self.L):
            sh1, sc1, g1, sh2, sc2, g2 = self._mod(f"w_mod.{l}", f"b_mod.{l}", cvecs, 6)
            h = self.norm(z) * (1.0 + sc1) + sh1
            qkv = h @ self.w[f"w_qkv.{l}"] + self.w[f"b_qkv.{l}"]
            q = self.rope(self._heads(qkv[:, :self.d]), fr, r, c)
            kk = self.rope(self._heads(qkv[:, self.d:2 * self.d]), fr, r, c)
            vv = self._heads(qkv[:, 2 * self.d:])
            newK.append(kk)
            newV.append(vv)
            if store:
                for j in range(k):
                    self.kv[l][base + j] = (kk[:, j * T:(j + 1) * T].copy(), vv[:, j * T:(j + 1) * T].copy())
            if kv_only_last and l == self.L - 1:
                break
            o = np.empty((k * T, self.d), F64)
            for j in range(k):
                f = base + j
                ks, vs = [], []
                for g in range(max(0, f - self.W), f + 1):
                    if g >= base:
                        ks.append(kk[:, (g - base) * T:(g - base + 1) * T])
                        vs.append(vv[:, (g - base) * T:(g - base + 1) * T])
                    else:
                        ks.append(self.kv[l][g][0])
                        vs.append(self.kv[l][g][1])
                Kc, Vc = np.concatenate(ks, axis=1), np.concatenate(vs, axis=1)
                S = q[:, j * T:(j + 1) * T] @ Kc.transpose(0, 2, 1) / math.sqrt(self.dh)
                o[j * T:(j + 1) * T] = (softmax_rows(S) @ Vc).transpose(1, 0, 2).reshape(T, self.d)
            z = z + g1 * (o @ self.w[f"w_o.{l}"] + self.w[f"b_o.{l}"])
            h = self.norm(z) * (1.0 + sc2) + sh2
            m = mlp(h, self.w[f"w_fc1.{l}"], self.w[f"b_fc1.{l}"], self.w[f"w_fc2.{l}"], self.w[f"b_fc2.{l}"],
                    self.cfg.get("act", 0))
            z = z + g2 * m
        if kv_only_last:
            return None, newK, newV
        return self._final(z, cvecs), newK, newV

    # ---------------- the calls of the boundary ----------------
    def denoise_step(self, x_t, t: float, action: int, offset: int = 0):
        """One forward pass over k in-flight frames that follow the cached
        (committed + tentative) frames; `offset` in-flight frames of earlier
        calls are kept as context.  Returns the velocity [k,C,H,W]."""
        k = x_t.shape[0]
        assert 1 <= k and offset + k <= self.kmax
        v, _, _ = self.forward_chunk(np.asarray(x_t, F64), [t] * k, [action] * k, self.n_total + offset)
        return v

    def _commit(self, x0, actions, ctx_noise, tentative: bool):
        n = x0.shape[0]
        tp = float(self.cfg["t_ctx_trig"])
        z = np.zeros_like(np.asarray(x0, F64)) if ctx_noise is None else np.asarray(ctx_noise, F64)
        x_trig = renoise(x0, z, tp, self.sigma_d)           # Section 4.3: perturb the context frames
        x_in = fm_input(x_trig, tp, self.sigma_d)
        self.forward_chunk(x_in, [fm_time(tp)] * n, list(actions), self.n_total, kv_only_last=True)
        if tentative:
            self.n_tentative += n
        else:
            self.n_committed += n
        self._evict()

    def commit_frame(self, x0, actions, ctx_noise=None):
        assert self.n_tentative == 0
        self._commit(x0, actions, ctx_noise, tentative=False)

    def _evict(self):
        lo = self.n_total - self.W - self.kmax
        for l in range(self.L):
            for f in [f for f in self.kv[l] if f < lo]:
                del self.kv[l][f]

    def speculate(self, k: int, action: int, noise, ctx_noise=None):
        """Section 4.1 "Sampling" + Section 4.2: S denoise/re-noise steps over
        k frames decoded together under `action`, then the k clean frames are
        appended to the cache as tentative.  noise [S,k,C,H,W].  Returns x0."""
        S = self.cfg["n_steps"]
        sched = trig_schedule(S)
        noise = np.asarray(noise, F64)
        x = self.sigma_d * noise[0]
        x0 = None
        for s in range(S):
            tp = sched[s]
            t = fm_time(tp)
            x_in = fm_input(x, tp, self.sigma_d)
            v = self.denoise_step(x_in, t, action)
            x0 = f_theta(x, F_theta(x_in, v, t), tp, self.sigma_d)
            if s + 1 < S:
                x = renoise(x0, noise[s + 1], sched[s + 1], self.sigma_d)
        self._commit(x0, [action] * k, ctx_noise, tentative=True)
        return x0

    def sample_dpmpp(self, k: int, action: int, noise, n_evals: int = 18, ctx_noise=None):
        """The undistilled sampler of Section 3.2 "Sampling": the Flow-Matching model integrated from pure noise
        with DPM-Solver++ (n_evals function evaluations, 18 in the paper's experiments) for k frames decoded
        together under `action`; the clean frames are appended to the cache as tentative.  noise [k,C,H,W] in
        unit variance; latents are in units of sigma_d, so the model sees x/sigma_d.  Data prediction from the
        velocity: x0 = x_t - t v (Section 3.2).  Returns x0 [k,C,H,W]."""
        def x0_fn(x, t):
            return x - t * self.denoise_step(x, t, action)
        x0 = self.sigma_d * dpmpp_2m(x0_fn, np.asarray(noise, F64), n_evals)
        self._commit(x0, [action] * k, ctx_noise, tentative=True)
        return x0

    def rollback(self, n_accept: int):
        """Keep the first n_accept tentative frames, drop the rest."""
        assert 0 <= n_accept <= self.n_tentative
        keep = self.n_committed + n_accept
        for l in range(self.L):
            for f in [f for f in self.kv[l] if f >= keep]:
                del self.kv[l][f]
        self.n_committed = keep
        self.n_tentative = 0

    def kv_frame(self, layer: int, frame: int):
        return self.kv[layer][frame]

    def kv_digest(self) -> int:
        """Digest of the counters and of the K/V of the frames a future query
        can still see (the last W cached frames), in frame order."""
        h = zlib.crc32(struct.pack("<ii", self.n_committed, self.n_tentative))
        for l in range(self.L):
            for f in range(self.window_first(), self.n_total):
                K, V = self.kv[l][f]
                h = zlib.crc32(np.ascontiguousarray(K).tobytes(), h)
                h = zlib.crc32(np.ascontiguousarray(V).tobytes(), h)
        return h

    def generate(self, true_actions, n_frames: int, k: int, noise_fn, ctx_noise_fn=None):
        """Speculative generation loop (appendix listing's control flow):
        frame i is generated under true_actions[i]; the k-1 further frames are
        generated under the same action and verified afterwards.
        noise_fn(i, k) -> [S,k,C,H,W]; ctx_noise_fn(i, k) -> [k,C,H,W] or None.
        Returns (frames list, speculated count, accepted count, passes)."""
        out = []
        spec = acc = passes = 0
        i = 0
        while i < n_frames:
            kk = min(k, n_frames - i)
            cn = None if ctx_noise_fn is None else ctx_noise_fn(i, kk)
            x0 = self.speculate(kk, int(true_actions[i]), noise_fn(i, kk), cn)
            n = accepted_count(true_actions[:n_frames], i, kk)
            self.rollback(n)
            out.extend(list(x0[:n]))
            spec += kk
            acc += n
            passes += 1
            i += n
        return out, spec, acc, passes


def attention_block_causal(q, k, v, q_frame, k_frame, window: int, return_probs: bool = False):
    """Block-wise causal attention written out with an explicit dense mask.
    q [H,nq,dh], k,v [H,nk,dh]; q_frame[nq], k_frame[nk] integer frame ids.
    Key j is visible to query i iff  q_frame[i]-window <= k_frame[j] <= q_frame[i]."""
    q, k, v = np.asarray(q, F64), np.asarray(k, F64), np.asarray(v, F64)
    qf, kf = np.asarray(q_frame), np.asarray(k_frame)
    allowed = (kf[None, :] <= qf[:, None]) & (kf[None, :] >= qf[:, None] - window)
    S = q @ k.transpose(0, 2, 1) / math.sqrt(q.shape[-1]) + np.where(allowed, 0.0, -np.inf)[None]
    Pm = softmax_rows(S)
    o = Pm @ v
    return (o, Pm) if return_probs else o
