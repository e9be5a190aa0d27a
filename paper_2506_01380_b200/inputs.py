"""Seeded synthetic inputs for the block-causal DiT hot path.

This module holds configuration tables and random-tensor generators only.  It
contains none of the method's arithmetic: both the CUDA library's tests and the
CPU oracle's tests draw their weights, latents, noise and action chains from
here so that the two sides see identical data.

Shapes follow the paper's workload (Section 5, "Dataset and Preprocessing":
384x224 frames -> 24x14 = 336 latent tokens per frame, 16-frame evaluation
context, 32-frame training context) and Appendix Table "configuration of
different size of models" for the paper-exact sizes.
"""
from __future__ import annotations

import numpy as np

# dtype codes shared with the C ABI (nfd_cfg.dtype)
DTYPE_FP32 = 0
DTYPE_BF16 = 1


def _base_cfg(**kw):
    cfg = dict(
        n_layers=2, d_model=128, n_heads=4, head_dim=32, d_mlp=512,
        latent_c=4, latent_h=8, latent_w=8, patch=1,
        n_actions=8, ctx_frames=4, max_spec=4, n_streams=1,
        dtype=DTYPE_FP32, norm=0, act=0,
        rope_t=8, rope_h=12, rope_w=12,
        rope_theta=10000.0, norm_eps=1e-6, t_scale=1000.0,
        sigma_d=0.5, t_ctx_trig=0.1, n_steps=4,
    )
    cfg.update(kw)
    return cfg


def make_cfg(name: str, **overrides) -> dict:
    """Named configurations.

    tiny      2 layers, d=128, 4 heads x 32, MLP 512, 64 tokens/frame, fp32.
    attn      the 16-head x 64 attention shape embedded in a 1-layer model.
    nfd310m   24 layers, d=1024, 16 heads x 64, MLP 4096, 336 tokens/frame, bf16.
    paper130m / paper310m / paper774m: the sizes printed in the paper's appendix
              table (hidden, MLP, heads, layers); GELU MLP unless act=1 is passed
              (gated MLP, the reading that the 8/3 MLP width suggests).
    tiny_gated / tiny_gated_bf16: the tiny model with a gated MLP of width 340
              (not a multiple of 8, like the 2730 of the paper's 310M model).
    """
    if name == "tiny":
        cfg = _base_cfg()
    elif name == "tiny_bf16":
        cfg = _base_cfg(dtype=DTYPE_BF16)
    elif name == "tiny_gated":
        cfg = _base_cfg(act=1, d_mlp=340)
    elif name == "tiny_gated_bf16":
        cfg = _base_cfg(act=1, d_mlp=340, dtype=DTYPE_BF16)
    elif name == "nfd310m":
        cfg = _base_cfg(
            n_layers=24, d_model=1024, n_heads=16, head_dim=64, d_mlp=4096,
            latent_c=16, latent_h=48, latent_w=28, patch=2,
            n_actions=32, ctx_frames=16, max_spec=4, n_streams=1,
            dtype=DTYPE_BF16, rope_t=16, rope_h=24, rope_w=24)
    elif name == "nfd310m_slice":      # 2-layer slice of the 310M-class shape
        cfg = make_cfg("nfd310m", n_layers=2)
    elif name == "nfd310m_b8":
        cfg = make_cfg("nfd310m", ctx_frames=32, n_streams=8)
    elif name == "paper130m":
        cfg = make_cfg("nfd310m", n_layers=12, d_model=768, n_heads=12, d_mlp=2048)
    elif name == "paper310m":
        cfg = make_cfg("nfd310m", n_layers=16, d_model=1024, n_heads=16, d_mlp=2730)
    elif name == "paper774m":
        cfg = make_cfg("nfd310m", n_layers=18, d_model=1536, n_heads=24, d_mlp=4096)
    else:
        raise KeyError(name)
    cfg.update(overrides)
    return cfg


def tokens_per_frame(cfg) -> int:
    return (cfg["latent_h"] // cfg["patch"]) * (cfg["latent_w"] // cfg["patch"])


def patch_len(cfg) -> int:
    return cfg["latent_c"] * cfg["patch"] * cfg["patch"]


def frame_shape(cfg):
    return (cfg["latent_c"], cfg["latent_h"], cfg["latent_w"])


def round_bf16(a: np.ndarray) -> np.ndarray:
    """Round an fp32 array to the nearest bf16 value (ties to even), kept as fp32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).copy()
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    lsb += np.uint32(0x7FFF)
    u += lsb                      # finite inputs cannot overflow 32 bits here
    u &= np.uint32(0xFFFF0000)
    return u.view(np.float32).reshape(a.shape)


def weight_shapes(cfg) -> dict:
    """Name -> shape of every parameter, all row-major [in, out]."""
    d, dm, P = cfg["d_model"], cfg["d_mlp"], patch_len(cfg)
    shapes = {
        "w_pe": (P, d), "b_pe": (d,),
        "w_t1": (256, d), "b_t1": (d,),
        "w_t2": (d, d), "b_t2": (d,),
        "a_emb": (cfg["n_actions"], d),
        "w_fmod": (d, 2 * d), "b_fmod": (2 * d,),
        "w_out": (d, P), "b_out": (P,),
    }
    for l in range(cfg["n_layers"]):
        shapes[f"w_mod.{l}"] = (d, 6 * d)
        shapes[f"b_mod.{l}"] = (6 * d,)
        shapes[f"w_qkv.{l}"] = (d, 3 * d)
        shapes[f"b_qkv.{l}"] = (3 * d,)
        shapes[f"w_o.{l}"] = (d, d)
        shapes[f"b_o.{l}"] = (d,)
        # act 1 (gated MLP): gate and up projections side by side
        shapes[f"w_fc1.{l}"] = (d, dm * (2 if cfg.get("act", 0) == 1 else 1))
        shapes[f"b_fc1.{l}"] = (dm * (2 if cfg.get("act", 0) == 1 else 1),)
        shapes[f"w_fc2.{l}"] = (dm, d)
        shapes[f"b_fc2.{l}"] = (d,)
    return shapes


def make_weights(cfg, seed: int = 0, kind: str = "paper") -> dict:
    """Seeded random-init weights as fp32 numpy arrays.

    kind="paper":  every matrix and bias N(0, 0.02^2).
    kind="stress": matrices N(0, 1/fan_in), biases N(0, 0.1^2), and the gate
                   chunks of every modulation bias set to 1 so that each
                   residual branch contributes at full strength.
    Values are rounded to bf16 when cfg["dtype"] is bf16 so that the fp64
    oracle and the bf16 device path start from the same numbers.
    """
    rng = np.random.default_rng(seed)
    d = cfg["d_model"]
    out = {}
    for name, shape in weight_shapes(cfg).items():
        if kind == "paper":
            w = rng.standard_normal(shape, dtype=np.float32) * np.float32(0.02)
        elif kind == "stress":
            if len(shape) == 2 and name != "a_emb":
                w = rng.standard_normal(shape, dtype=np.float32) * np.float32(1.0 / np.sqrt(shape[0]))
            elif name == "a_emb":
                w = rng.standard_normal(shape, dtype=np.float32)
            else:
                w = rng.standard_normal(shape, dtype=np.float32) * np.float32(0.1)
                if name.startswith("b_mod."):
                    w[2 * d:3 * d] = 1.0
                    w[5 * d:6 * d] = 1.0
        else:
            raise KeyError(kind)
        if cfg["dtype"] == DTYPE_BF16:
            w = round_bf16(w)
        out[name] = np.ascontiguousarray(w, dtype=np.float32)
    return out


def make_latents(cfg, n_frames: int, seed: int) -> np.ndarray:
    """N(0,1) latent frames [n, C, H, W], fp32."""
    rng = np.random.default_rng(seed)
    return rng.standard_normal((n_frames,) + frame_shape(cfg), dtype=np.float32)


def make_noise(cfg, n_steps: int, k: int, seed: int) -> np.ndarray:
    """N(0,1) sampler noise [n_steps, k, C, H, W], fp32."""
    rng = np.random.default_rng(seed)
    return rng.standard_normal((n_steps, k) + frame_shape(cfg), dtype=np.float32)


def make_actions_uniform(cfg, n: int, seed: int) -> np.ndarray:
    rng = np.random.default_rng(seed)
    return rng.integers(0, cfg["n_actions"], size=n, dtype=np.int64).astype(np.int32)


def make_action_chain(cfg, n: int, seed: int, p_repeat: float = 0.8) -> np.ndarray:
    """Markov chain over the action alphabet: a[0] uniform; a[i+1] = a[i] with
    probability p_repeat, otherwise uniform over the other n_actions-1 symbols."""
    rng = np.random.default_rng(seed)
    A = cfg["n_actions"]
    a = np.empty(n, dtype=np.int32)
    a[0] = rng.integers(0, A)
    for i in range(1, n):
        if rng.random() < p_repeat:
            a[i] = a[i - 1]
        else:
            a[i] = (a[i - 1] + 1 + rng.integers(0, A - 1)) % A
    return a


def make_qkv(n_heads: int, head_dim: int, n_q: int, n_k: int, seed: int, bf16: bool = True):
    """N(0,1) Q [H, n_q, dh], K and V [H, n_k, dh] for the attention-only case."""
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((n_heads, n_q, head_dim), dtype=np.float32)
    k = rng.standard_normal((n_heads, n_k, head_dim), dtype=np.float32)
    v = rng.standard_normal((n_heads, n_k, head_dim), dtype=np.float32)
    if bf16:
        q, k, v = round_bf16(q), round_bf16(k), round_bf16(v)
    return q, k, v
