"""Small, self-ending workload for profiler captures of libnfd's kernels.

    python -m paper_2506_01380_b200.profile_case [--layers 2] [--ctx 16] [--k 1] [--passes 2] [--no-graph]

Builds the 310M-class shape with a reduced number of layers (so the device holds
well under a GB), fills the KV context with commit passes and runs a few
denoising passes.  Meant to be wrapped by `ncu -k regex:... -c N`.
"""
from __future__ import annotations

import argparse

import torch

from . import inputs as I
from .nfd import NFD


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=2)
    ap.add_argument("--ctx", type=int, default=16)
    ap.add_argument("--k", type=int, default=1)
    ap.add_argument("--passes", type=int, default=2)
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-fast", action="store_true")
    a = ap.parse_args()
    cfg = I.make_cfg("nfd310m", n_layers=a.layers, ctx_frames=a.ctx)
    dev = torch.device("cuda:0")
    g = torch.Generator(device=dev)
    g.manual_seed(0)
    w = {n: torch.randn(s, generator=g, device=dev) * 0.02 for n, s in I.weight_shapes(cfg).items()}
    nfd = NFD(cfg, w)
    if a.no_graph:
        nfd.set_option("graph", 0)
    if a.no_fast:
        nfd.set_option("fast", 0)
    fs = I.frame_shape(cfg)
    for i in range(0, a.ctx, 4):
        n = min(4, a.ctx - i)
        nfd.commit_frame(torch.randn((n,) + fs, generator=g, device=dev), [1] * n)
    x = torch.randn((a.k,) + fs, generator=g, device=dev)
    for _ in range(a.passes):
        v = nfd.denoise_step(x, 0.7, 3)
    torch.cuda.synchronize()
    assert nfd.status() == 0
    print("ok", float(v.abs().mean()))


if __name__ == "__main__":
    main()
