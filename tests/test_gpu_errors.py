"""Error paths of libnfd on the GPU, each made without a device fault: a launch that
the runtime refuses on the host, a pass descriptor with a bad index that the first
kernel of the pass catches, and a bounded device-side wait that runs out because the
producer left one pipeline stage out.  After each, the context must keep working and
give bitwise the results of a context that never saw the error."""
import numpy as np
import pytest

from paper_2506_01380_b200 import inputs as I

pytestmark = pytest.mark.gpu

E_CUDA, E_TIMEOUT, E_DEVICE = -7, -8, -9


def _pair(name="tiny_bf16", seed=13):
    import torch
    from paper_2506_01380_b200.nfd import NFD
    cfg = I.make_cfg(name)
    w = I.make_weights(cfg, seed, "stress")
    a, b = NFD(cfg, w), NFD(cfg, w)
    x0 = torch.as_tensor(I.make_latents(cfg, 2, 1)).cuda()
    for g in (a, b):
        g.commit_frame(x0, [1, 2])
    return cfg, a, b, torch


def _same_generation(cfg, a, b, torch, seed):
    noise = torch.as_tensor(I.make_noise(cfg, cfg["n_steps"], 2, seed)).cuda()
    ya, yb = a.speculate(2, 3, noise), b.speculate(2, 3, noise)
    assert torch.equal(ya, yb)
    a.rollback(1), b.rollback(1)
    assert a.kv_state() == b.kv_state() and a.kv_hash() == b.kv_hash()
    assert a.status() == 0 and b.status() == 0


@pytest.mark.parametrize("graph", [1, 0])
def test_refused_launch_fails_one_call_only(graph):
    from paper_2506_01380_b200.nfd import NfdError
    cfg, a, b, torch = _pair()
    a.set_option("graph", graph), b.set_option("graph", graph)
    noise = torch.as_tensor(I.make_noise(cfg, cfg["n_steps"], 2, 5)).cuda()
    s0 = a.kv_state()
    a.set_option("test_fail_launch", 1)
    with pytest.raises(NfdError) as e:
        a.speculate(2, 3, noise)
    assert e.value.code == E_CUDA
    assert a.kv_state() == s0, "a failed call must not count frames"
    assert a.status() == 0                       # a host-side refusal: nothing ran wrongly on the device
    _same_generation(cfg, a, b, torch, 6)        # the very next call works, and so do the ones after it
    _same_generation(cfg, a, b, torch, 7)


def test_bad_descriptor_is_caught_on_the_device():
    cfg, a, b, torch = _pair()
    x = torch.as_tensor(I.make_latents(cfg, 1, 3)).cuda()
    a.set_option("test_corrupt_desc", 1)
    a.denoise_step(x, 0.5, 1)                    # enqueued; the device finds the bad batch slot
    assert a.status() == E_DEVICE
    assert a.status() == E_DEVICE                # the latch keeps the code ...
    a.set_option("clear_status", 1)              # ... until it is cleared
    assert a.status() == 0
    # the redirected pass wrote into slot 0's pages: start both contexts afresh and compare
    x0 = torch.as_tensor(I.make_latents(cfg, 2, 1)).cuda()
    for g in (a, b):
        g.reset(0)
        g.commit_frame(x0, [1, 2])
    _same_generation(cfg, a, b, torch, 8)


@pytest.mark.parametrize("name", ["tiny_bf16", "nfd310m_slice"])
def test_expired_wait_surfaces_as_timeout_and_context_survives(name):
    """Every tensor-core GEMM's producer leaves out its last stage; the consumer's wait (limit shortened to
    200 microseconds) gives up, latches NFD_E_TIMEOUT and the kernel leaves by its normal exit."""
    cfg, a, b, torch = _pair(name)
    x = torch.as_tensor(I.make_latents(cfg, 1, 3)).cuda()
    a.set_option("test_wait_limit_us", 200)
    a.set_option("test_skip_stage", 1)
    a.denoise_step(x, 0.5, 1)
    assert a.status() == E_TIMEOUT
    a.set_option("test_skip_stage", 0)
    a.set_option("test_wait_limit_us", 0)
    a.set_option("clear_status", 1)
    assert a.status() == 0
    v1, v2 = a.denoise_step(x, 0.5, 1), b.denoise_step(x, 0.5, 1)
    assert torch.equal(v1, v2), "the context must compute as before once the switch is off"
    _same_generation(cfg, a, b, torch, 9)
