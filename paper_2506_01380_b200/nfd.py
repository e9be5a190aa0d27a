"""Thin ctypes binding of libnfd (include/nfd.h).

Argument marshalling only: every step of the forward pass, the sampler, the
cache append and the rollback run inside the CUDA library.  torch is used for
device memory and for the CUDA stream handed to the library.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

from . import inputs as I

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libnfd.so")
_lib = None

CFG_INT_FIELDS = ["n_layers", "d_model", "n_heads", "head_dim", "d_mlp", "latent_c", "latent_h", "latent_w", "patch",
                  "n_actions", "ctx_frames", "max_spec", "n_streams", "dtype", "norm", "act",
                  "rope_t", "rope_h", "rope_w"]
CFG_FLOAT_FIELDS = ["rope_theta", "norm_eps", "t_scale", "sigma_d", "t_ctx_trig"]


class NfdCfg(C.Structure):
    _fields_ = ([(n, C.c_int) for n in CFG_INT_FIELDS] + [(n, C.c_float) for n in CFG_FLOAT_FIELDS]
                + [("n_steps", C.c_int)])


_SINGLE = ["w_pe", "b_pe", "w_t1", "b_t1", "w_t2", "b_t2", "a_emb"]
_LAYER = ["w_mod", "b_mod", "w_qkv", "b_qkv", "w_o", "b_o", "w_fc1", "b_fc1", "w_fc2", "b_fc2"]
_TAIL = ["w_fmod", "b_fmod", "w_out", "b_out"]


class NfdWeights(C.Structure):
    _fields_ = ([(n, C.c_void_p) for n in _SINGLE] + [(n, C.POINTER(C.c_void_p)) for n in _LAYER]
                + [(n, C.c_void_p) for n in _TAIL])


EXPORTS = ["nfd_create", "nfd_destroy", "nfd_reset", "nfd_denoise_step", "nfd_denoise_step_at",
           "nfd_denoise_step_batched", "nfd_commit_frame", "nfd_speculate", "nfd_speculate_batched",
           "nfd_rollback", "nfd_kv_state", "nfd_kv_hash", "nfd_kv_read", "nfd_attention", "nfd_status",
           "nfd_launch_count", "nfd_set_option", "nfd_warm_modulation", "nfd_strerror", "nfd_profile_begin",
           "nfd_profile_end",
           "nfd_profile_class_count", "nfd_profile_class_name", "nfd_attention_noalloc", "nfd_cond_cache_stats",
           "nfd_sample_dpmpp", "nfd_accepted_count", "nfd_debug_read"]


class NfdError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        msg = load().nfd_strerror(code).decode() if _lib is not None else ""
        super().__init__(f"{what} failed: {code} ({msg})")


def load():
    """Load libnfd.so (built in-tree by paper_2506_01380_b200.build).  There is no
    fallback of any kind: a missing library is an error."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} is missing: run `python -m paper_2506_01380_b200.build` "
                           "(needs nvcc); libnfd has no CPU or PyTorch fallback")
    lib = C.CDLL(_LIB_PATH)
    vp, ip, fp = C.c_void_p, C.POINTER(C.c_int), C.POINTER(C.c_float)
    lib.nfd_create.argtypes = [C.POINTER(vp), C.POINTER(NfdWeights), C.POINTER(NfdCfg), vp]
    lib.nfd_destroy.argtypes = [vp]
    lib.nfd_reset.argtypes = [vp, C.c_int]
    lib.nfd_denoise_step.argtypes = [vp, C.c_int, vp, C.c_int, C.c_float, C.c_int, vp]
    lib.nfd_denoise_step_at.argtypes = [vp, C.c_int, C.c_int, vp, C.c_int, C.c_float, C.c_int, vp]
    lib.nfd_denoise_step_batched.argtypes = [vp, C.c_int, ip, vp, C.c_int, fp, ip, vp]
    lib.nfd_commit_frame.argtypes = [vp, C.c_int, vp, C.c_int, ip, vp]
    lib.nfd_speculate.argtypes = [vp, C.c_int, C.c_int, C.c_int, vp, vp, vp]
    lib.nfd_speculate_batched.argtypes = [vp, C.c_int, ip, C.c_int, ip, vp, vp, vp]
    lib.nfd_sample_dpmpp.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.c_int, vp, vp, vp]
    lib.nfd_rollback.argtypes = [vp, C.c_int, C.c_int]
    lib.nfd_kv_state.argtypes = [vp, C.c_int, ip, ip, ip]
    lib.nfd_kv_hash.argtypes = [vp, C.c_int, C.POINTER(C.c_ulonglong)]
    lib.nfd_kv_read.argtypes = [vp, C.c_int, C.c_int, C.c_int, vp, vp]
    lib.nfd_attention.argtypes = [vp, vp, vp, vp, C.c_int, C.c_int, C.c_int, vp]
    lib.nfd_status.argtypes = [vp]
    lib.nfd_launch_count.argtypes = [vp]
    lib.nfd_launch_count.restype = C.c_longlong
    lib.nfd_set_option.argtypes = [vp, C.c_char_p, C.c_int]
    lib.nfd_warm_modulation.argtypes = [vp]
    lib.nfd_profile_begin.argtypes = [vp]
    lib.nfd_profile_end.argtypes = [vp, C.c_int, C.POINTER(C.c_longlong), fp]
    lib.nfd_profile_class_count.argtypes = []
    lib.nfd_profile_class_name.argtypes = [C.c_int]
    lib.nfd_profile_class_name.restype = C.c_char_p
    lib.nfd_attention_noalloc.argtypes = [vp, vp, vp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                          vp, vp]
    lib.nfd_cond_cache_stats.argtypes = [vp, C.POINTER(C.c_longlong), C.POINTER(C.c_longlong)]
    lib.nfd_accepted_count.argtypes = [ip, C.c_int, C.c_int, C.c_int]
    lib.nfd_debug_read.argtypes = [vp, C.c_char_p, vp, C.c_longlong]
    lib.nfd_strerror.argtypes = [C.c_int]
    lib.nfd_strerror.restype = C.c_char_p
    _lib = lib
    return lib


def make_c_cfg(cfg: dict) -> NfdCfg:
    c = NfdCfg()
    for n in CFG_INT_FIELDS + ["n_steps"]:
        setattr(c, n, int(cfg[n]))
    for n in CFG_FLOAT_FIELDS:
        setattr(c, n, float(cfg[n]))
    return c


def _ints(v):
    a = (C.c_int * len(v))(*[int(x) for x in v])
    return a


def _floats(v):
    return (C.c_float * len(v))(*[float(x) for x in v])


def _check(code: int, what: str):
    if code != 0:
        raise NfdError(code, what)


def accepted_frames(true_actions, i: int, k: int) -> int:
    """nfd_accepted_count: how many of the frames i .. i+k-1, generated under
    true_actions[i], were generated under their own true action; pass it to rollback()."""
    n = len(true_actions)
    r = load().nfd_accepted_count(_ints(true_actions), n, int(i), int(k))
    _check(0 if r > 0 else (r or -4), "nfd_accepted_count")
    return r


def attention_noalloc(q, k_pages, v_pages, n_q_frames: int, window: int, out, stream=None):
    """nfd_attention_noalloc: block-causal attention without a context and without
    any allocation (the caller passes `out`).  For hosts that may not call
    cudaMalloc where they need attention (inside a stream capture, in a frame
    loop that bans allocator calls, under a foreign memory arena).
    q [H, n_q*T, dh]; k_pages, v_pages [n_kv, H, T, dh]; out [n_q*T, H*dh];
    all on one device, same dtype (float32 or bfloat16), contiguous."""
    lib = load()
    n_kv, H, T, dh = k_pages.shape
    dtype = I.DTYPE_BF16 if q.dtype == torch.bfloat16 else I.DTYPE_FP32
    for t in (q, k_pages, v_pages, out):
        assert t.is_cuda and t.is_contiguous() and t.dtype == q.dtype
    assert tuple(q.shape) == (H, n_q_frames * T, dh) and tuple(out.shape) == (n_q_frames * T, H * dh)
    st = torch.cuda.current_stream(q.device) if stream is None else stream
    _check(lib.nfd_attention_noalloc(C.c_void_p(q.data_ptr()), C.c_void_p(k_pages.data_ptr()),
                                     C.c_void_p(v_pages.data_ptr()), dtype, H, dh, T, n_q_frames, n_kv, window,
                                     C.c_void_p(out.data_ptr()), C.c_void_p(st.cuda_stream)),
           "nfd_attention_noalloc")
    return out


class NFD:
    """One libnfd context on one GPU.  Method names and arguments follow the C ABI."""

    def __init__(self, cfg: dict, weights: dict, device: str = "cuda:0"):
        if not torch.cuda.is_available():
            raise RuntimeError("libnfd needs a CUDA device; there is no CPU path")
        self.lib = load()
        self.cfg = dict(cfg)
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.tdtype = torch.bfloat16 if cfg["dtype"] == I.DTYPE_BF16 else torch.float32
        self.stream = torch.cuda.Stream(device=self.device)
        self.frame_shape = I.frame_shape(cfg)
        self.T = I.tokens_per_frame(cfg)
        self._h = C.c_void_p()
        # upload the caller's weights in the storage type; the library copies / repacks them
        dev = {k: torch.as_tensor(np.ascontiguousarray(v)).to(self.device, self.tdtype).contiguous()
               if not torch.is_tensor(v) else v.to(self.device, self.tdtype).contiguous()
               for k, v in weights.items()}
        w = NfdWeights()
        keep = []
        for n in _SINGLE + _TAIL:
            setattr(w, n, dev[n].data_ptr())
        for n in _LAYER:
            arr = (C.c_void_p * cfg["n_layers"])(*[dev[f"{n}.{l}"].data_ptr() for l in range(cfg["n_layers"])])
            keep.append(arr)
            setattr(w, n, C.cast(arr, C.POINTER(C.c_void_p)))
        torch.cuda.synchronize(self.device)
        ccfg = make_c_cfg(cfg)
        _check(self.lib.nfd_create(C.byref(self._h), C.byref(w), C.byref(ccfg), C.c_void_p(self.stream.cuda_stream)),
               "nfd_create")
        del dev, keep

    # -- stream hand-off between torch's current stream and the library's stream
    def _enter(self):
        cur = torch.cuda.current_stream(self.device)
        if cur != self.stream:
            self.stream.wait_stream(cur)

    def _exit(self):
        cur = torch.cuda.current_stream(self.device)
        if cur != self.stream:
            cur.wait_stream(self.stream)

    def _f32(self, x, shape=None):
        assert torch.is_tensor(x) and x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()
        if shape is not None:
            assert tuple(x.shape) == tuple(shape), (tuple(x.shape), tuple(shape))
        return C.c_void_p(x.data_ptr())

    def close(self):
        if self._h:
            self.lib.nfd_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self, stream: int = 0):
        _check(self.lib.nfd_reset(self._h, stream), "nfd_reset")

    def denoise_step(self, x_t, t: float, action: int, stream: int = 0, offset: int = 0, out=None):
        k = x_t.shape[0]
        v = torch.empty_like(x_t) if out is None else out
        self._enter()
        _check(self.lib.nfd_denoise_step_at(self._h, stream, offset, self._f32(x_t, (k,) + self.frame_shape), k,
                                            float(t), int(action), self._f32(v)), "nfd_denoise_step")
        self._exit()
        return v

    def denoise_step_batched(self, streams, x_t, t, actions, out=None):
        n, k = x_t.shape[0], x_t.shape[1]
        v = torch.empty_like(x_t) if out is None else out
        self._enter()
        _check(self.lib.nfd_denoise_step_batched(self._h, n, _ints(streams), self._f32(x_t), k, _floats(t),
                                                 _ints(actions), self._f32(v)), "nfd_denoise_step_batched")
        self._exit()
        return v

    def commit_frame(self, x0, actions, ctx_noise=None, stream: int = 0):
        n = x0.shape[0]
        self._enter()
        _check(self.lib.nfd_commit_frame(self._h, stream, self._f32(x0, (n,) + self.frame_shape), n, _ints(actions),
                                         self._f32(ctx_noise, x0.shape) if ctx_noise is not None else None),
               "nfd_commit_frame")
        self._exit()

    def speculate(self, k: int, action: int, noise, ctx_noise=None, stream: int = 0, out=None):
        S = self.cfg["n_steps"]
        x0 = torch.empty((k,) + self.frame_shape, device=self.device, dtype=torch.float32) if out is None else out
        self._enter()
        _check(self.lib.nfd_speculate(self._h, stream, k, int(action), self._f32(noise, (S, k) + self.frame_shape),
                                      self._f32(ctx_noise, x0.shape) if ctx_noise is not None else None,
                                      self._f32(x0)), "nfd_speculate")
        self._exit()
        return x0

    def sample_dpmpp(self, k: int, action: int, noise, n_evals: int = 18, ctx_noise=None, stream: int = 0, out=None):
        x0 = torch.empty((k,) + self.frame_shape, device=self.device, dtype=torch.float32) if out is None else out
        self._enter()
        _check(self.lib.nfd_sample_dpmpp(self._h, stream, k, int(action), int(n_evals),
                                         self._f32(noise, (k,) + self.frame_shape),
                                         self._f32(ctx_noise, x0.shape) if ctx_noise is not None else None,
                                         self._f32(x0)), "nfd_sample_dpmpp")
        self._exit()
        return x0

    def speculate_batched(self, streams, k: int, actions, noise, ctx_noise=None, out=None):
        n, S = len(streams), self.cfg["n_steps"]
        x0 = torch.empty((n, k) + self.frame_shape, device=self.device, dtype=torch.float32) if out is None else out
        self._enter()
        _check(self.lib.nfd_speculate_batched(self._h, n, _ints(streams), k, _ints(actions),
                                              self._f32(noise, (S, n, k) + self.frame_shape),
                                              self._f32(ctx_noise, x0.shape) if ctx_noise is not None else None,
                                              self._f32(x0)), "nfd_speculate_batched")
        self._exit()
        return x0

    def rollback(self, n_accept: int, stream: int = 0):
        _check(self.lib.nfd_rollback(self._h, stream, n_accept), "nfd_rollback")

    def kv_state(self, stream: int = 0):
        a, b, c = C.c_int(), C.c_int(), C.c_int()
        _check(self.lib.nfd_kv_state(self._h, stream, C.byref(a), C.byref(b), C.byref(c)), "nfd_kv_state")
        return a.value, b.value, c.value

    def kv_hash(self, stream: int = 0) -> int:
        h = C.c_ulonglong()
        self._enter()
        _check(self.lib.nfd_kv_hash(self._h, stream, C.byref(h)), "nfd_kv_hash")
        return h.value

    def kv_read(self, layer: int, frame: int, stream: int = 0):
        shape = (self.cfg["n_heads"], self.T, self.cfg["head_dim"])
        k = torch.empty(shape, device=self.device, dtype=torch.float32)
        v = torch.empty(shape, device=self.device, dtype=torch.float32)
        self._enter()
        _check(self.lib.nfd_kv_read(self._h, stream, layer, frame, self._f32(k), self._f32(v)), "nfd_kv_read")
        self._exit()
        return k, v

    def attention(self, q, k, v, n_q_frames: int, n_kv_frames: int, window: int, out=None):
        """q [H, n_q*T, dh]; k, v [H, n_kv*T, dh] (or None to reuse the pages of the last call)."""
        assert q.dtype == self.tdtype and q.is_contiguous()
        o = torch.empty((n_q_frames * self.T, self.cfg["d_model"]), device=self.device, dtype=self.tdtype) \
            if out is None else out
        self._enter()
        _check(self.lib.nfd_attention(self._h, C.c_void_p(q.data_ptr()),
                                      C.c_void_p(k.data_ptr()) if k is not None else None,
                                      C.c_void_p(v.data_ptr()) if v is not None else None,
                                      n_q_frames, n_kv_frames, window, C.c_void_p(o.data_ptr())), "nfd_attention")
        self._exit()
        return o

    def debug_read(self, name: str, n_elems: int):
        """First n_elems elements of an activation buffer of the last pass, as fp32."""
        out = torch.empty(int(n_elems), device=self.device, dtype=torch.float32)
        self._enter()
        _check(self.lib.nfd_debug_read(self._h, name.encode(), C.c_void_p(out.data_ptr()), int(n_elems)),
               "nfd_debug_read")
        self._exit()
        return out

    def status(self) -> int:
        return self.lib.nfd_status(self._h)

    def launch_count(self) -> int:
        return self.lib.nfd_launch_count(self._h)

    def cond_cache_stats(self):
        """(hits, misses) of the modulation cache since creation."""
        h, m = C.c_longlong(), C.c_longlong()
        _check(self.lib.nfd_cond_cache_stats(self._h, C.byref(h), C.byref(m)), "nfd_cond_cache_stats")
        return int(h.value), int(m.value)

    def profile_begin(self):
        _check(self.lib.nfd_profile_begin(self._h), "nfd_profile_begin")

    def profile_end(self) -> dict:
        """{class name: (launches, total milliseconds)}"""
        n = self.lib.nfd_profile_class_count()
        cnt, ms = (C.c_longlong * n)(), (C.c_float * n)()
        _check(self.lib.nfd_profile_end(self._h, n, cnt, ms), "nfd_profile_end")
        return {self.lib.nfd_profile_class_name(i).decode(): (int(cnt[i]), float(ms[i])) for i in range(n)}

    def warm_modulation(self) -> int:
        """Precompute the modulation of every (schedule time, action) pair; returns the number computed."""
        self._enter()
        try:
            n = self.lib.nfd_warm_modulation(self._h)
        finally:
            self._exit()
        if n < 0:
            _check(n, "nfd_warm_modulation")
        return n

    def set_option(self, name: str, value: int):
        _check(self.lib.nfd_set_option(self._h, name.encode(), int(value)), "nfd_set_option")
