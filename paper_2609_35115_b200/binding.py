"""ctypes binding with the same names as include/dc.h."""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libdc.so")
_lib = None

DC_MAX_CONV, DC_MAX_UP, DC_MAX_RES = 32, 4, 4
PIPE = {"conv": 1, "flow": 2, "vocoder": 3, "token2wav": 4}
PREC = {"f32": 0, "bf16": 1}
STATUS = {0: "DC_OK", 1: "DC_ERR_ARG", 2: "DC_ERR_CONFIG", 3: "DC_ERR_FRAMES", 4: "DC_ERR_OOM",
          5: "DC_ERR_CUDA", 6: "DC_ERR_TIMEOUT", 7: "DC_ERR_STATE"}

EXPORTS = ["dc_weights_count", "dc_create", "dc_destroy", "dc_stream_open", "dc_stream_reset",
           "dc_stream_close", "dc_decode_chunk", "dc_decode_batch", "dc_decode_chunk_host",
           "dc_stream_carry_info", "dc_get_counters", "dc_status_str", "dc_last_error",
           "dc_decode_batch_host", "dc_profile_begin", "dc_profile_end", "dc_conv_stack_noalloc",
           "dc_selftest_bounded_wait", "dc_stream_snapshot", "dc_stream_restore", "dc_snapshot_free",
           "dc_decode_wavefront", "dc_decode_wavefront_batch", "dc_stream_check_guards", "dc_test_fail_allocation", "dc_measure_fp32_peak"]


class dc_config(C.Structure):
    _fields_ = [("size", C.c_uint32), ("pipeline", C.c_int32), ("precision", C.c_int32),
                ("hidden", C.c_int32), ("n_conv", C.c_int32), ("dilations", C.c_int32 * DC_MAX_CONV),
                ("n_attn", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32),
                ("kv_cap", C.c_int32), ("n_steps", C.c_int32), ("f_chunk", C.c_int32),
                ("mel_dim", C.c_int32), ("n_up", C.c_int32), ("up_strides", C.c_int32 * DC_MAX_UP),
                ("up_channels", C.c_int32 * (DC_MAX_UP + 1)), ("n_res", C.c_int32),
                ("res_dilations", C.c_int32 * DC_MAX_RES), ("n_fft", C.c_int32), ("hop", C.c_int32),
                ("rms_eps", C.c_float), ("logmag_clamp", C.c_float), ("max_batch", C.c_int32),
                ("f_prompt", C.c_int32), ("f_lookahead", C.c_int32), ("noise_seed_lo", C.c_uint32), ("noise_seed_hi", C.c_uint32),
                ("cfg_scale", C.c_float), ("max_wave_frames", C.c_int32), ("options", C.c_uint32),
                ("excitation_std", C.c_float), ("excitation_seed_lo", C.c_uint32), ("excitation_seed_hi", C.c_uint32)]


class DCError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = load_library().dc_last_error().decode()
        super().__init__(f"{where}: {STATUS.get(status, status)} {msg}")


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Loads libdc.so; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} is missing: run `python -m paper_2609_35115_b200.build`")
    lib = C.CDLL(_LIB_PATH)
    vp, cp = C.c_void_p, C.POINTER
    lib.dc_weights_count.restype = C.c_size_t
    lib.dc_weights_count.argtypes = [cp(dc_config)]
    lib.dc_create.argtypes = [vp, C.c_size_t, cp(dc_config), cp(vp)]
    lib.dc_destroy.argtypes = [vp]
    lib.dc_stream_open.argtypes = [vp, cp(vp)]
    lib.dc_stream_reset.argtypes = [vp, vp]
    lib.dc_stream_snapshot.argtypes = [vp, cp(vp), vp]
    lib.dc_stream_restore.argtypes = [vp, vp, vp]
    lib.dc_snapshot_free.argtypes = [vp]
    lib.dc_stream_close.argtypes = [vp]
    lib.dc_decode_chunk.argtypes = [vp, vp, C.c_int, vp, cp(C.c_int), vp]
    lib.dc_decode_batch.argtypes = [vp, C.c_int, cp(vp), cp(vp), cp(C.c_int), cp(vp), vp]
    lib.dc_decode_wavefront.argtypes = [vp, vp, C.c_longlong, vp, cp(C.c_longlong), vp]
    lib.dc_decode_wavefront_batch.argtypes = [vp, C.c_int, cp(vp), cp(vp), cp(C.c_longlong), cp(vp), vp]
    lib.dc_decode_chunk_host.argtypes = [vp, vp, C.c_int, vp, cp(C.c_int), vp]
    lib.dc_decode_batch_host.argtypes = [vp, C.c_int, cp(vp), cp(vp), cp(C.c_int), cp(vp), vp]
    lib.dc_profile_begin.argtypes = [vp, C.c_int]
    lib.dc_profile_end.argtypes = [vp, cp(C.c_double), cp(C.c_uint64)]
    lib.dc_conv_stack_noalloc.argtypes = [vp, C.c_int, C.c_int, cp(C.c_int), vp, C.c_int, vp, vp]
    lib.dc_selftest_bounded_wait.argtypes = [C.c_int]
    lib.dc_stream_check_guards.argtypes = [vp, cp(C.c_int)]
    lib.dc_test_fail_allocation.argtypes = [C.c_int]
    lib.dc_measure_fp32_peak.argtypes = [cp(C.c_double)]
    lib.dc_stream_carry_info.argtypes = [vp, cp(C.c_uint64), C.c_int, cp(C.c_int)]
    lib.dc_get_counters.argtypes = [vp, cp(C.c_uint64)]
    lib.dc_status_str.restype = C.c_char_p
    lib.dc_status_str.argtypes = [C.c_int]
    lib.dc_last_error.restype = C.c_char_p
    lib.dc_last_error.argtypes = []
    for fn in EXPORTS:
        if fn not in ("dc_weights_count", "dc_status_str", "dc_last_error"):
            getattr(lib, fn).restype = C.c_int
    _lib = lib
    return lib


OPT_NO_GRAPH, OPT_NO_PDL, OPT_NO_ZEROCOPY, OPT_SERIAL_TAILS, OPT_ROUNDED_NORM, OPT_GUARD_ZONES = 1, 2, 4, 8, 16, 32
OPT_CTA_PAIRS = 64
OPT_SKIP_CONV_GEMM, OPT_SKIP_ATTENTION, OPT_EMPTY_KERNELS = 1 << 16, 1 << 17, 1 << 18     # measurement only: outputs are meaningless


def make_config(cfg, max_batch: int = 1, max_wave_frames: int = 0, options: int = 0) -> dc_config:
    """dc_workloads.DCConfig (or any object with the same attributes) -> dc_config."""
    c = dc_config()
    c.size = C.sizeof(dc_config)
    c.pipeline = PIPE[cfg.pipeline]
    c.precision = PREC[cfg.precision]
    c.hidden = cfg.hidden
    c.n_conv = len(cfg.dilations)
    for i, d in enumerate(cfg.dilations):
        c.dilations[i] = d
    c.n_attn, c.n_heads, c.head_dim, c.kv_cap = cfg.n_attn_layers, cfg.n_heads, cfg.head_dim, cfg.kv_cap
    c.n_steps, c.f_chunk, c.mel_dim = cfg.n_steps, cfg.f_chunk, cfg.mel_dim
    if cfg.pipeline in ("vocoder", "token2wav"):
        c.n_up = len(cfg.up_strides)
        for i, s in enumerate(cfg.up_strides):
            c.up_strides[i] = s
        for i, ch in enumerate(cfg.up_channels):
            c.up_channels[i] = ch
        c.n_res = len(cfg.res_dilations)
        for i, d in enumerate(cfg.res_dilations):
            c.res_dilations[i] = d
        c.n_fft, c.hop = cfg.n_fft, cfg.hop
    c.rms_eps, c.logmag_clamp = cfg.rms_eps, cfg.logmag_clamp
    c.max_batch = max_batch
    c.max_wave_frames = max_wave_frames
    c.options = options
    c.excitation_std = float(getattr(cfg, "excitation_std", 0.0))
    eseed = int(getattr(cfg, "excitation_seed", 0))
    c.excitation_seed_lo, c.excitation_seed_hi = eseed & 0xFFFFFFFF, (eseed >> 32) & 0xFFFFFFFF
    c.cfg_scale = float(getattr(cfg, "cfg_scale", 0.0))
    c.f_prompt = int(getattr(cfg, "f_prompt", 0))
    c.f_lookahead = int(getattr(cfg, "f_lookahead", 0))
    seed = int(getattr(cfg, "noise_seed", 0))
    c.noise_seed_lo, c.noise_seed_hi = seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF
    return c


def _check(status: int, where: str):
    if status != 0:
        raise DCError(status, where)


def _cuda_stream_handle(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


class Snapshot:
    def __init__(self, lib, handle):
        self.lib, self.handle = lib, handle

    def free(self):
        if self.handle:
            _check(self.lib.dc_snapshot_free(self.handle), "dc_snapshot_free")
            self.handle = None


class Model:
    """dc_create / dc_destroy."""

    def __init__(self, cfg, weights: np.ndarray, max_batch: int = 1, max_wave_frames: int = 0, options: int = 0):
        self.lib = load_library()
        self.cfg = cfg
        self.c_cfg = make_config(cfg, max_batch, max_wave_frames, options)
        w = np.ascontiguousarray(weights, dtype=np.float32)
        self.handle = C.c_void_p()
        _check(self.lib.dc_create(w.ctypes.data, w.size, C.byref(self.c_cfg), C.byref(self.handle)), "dc_create")
        self.out_per_frame = cfg.out_per_frame
        self.in_dim = cfg.in_dim

    def weights_count(self) -> int:
        return self.lib.dc_weights_count(C.byref(self.c_cfg))

    def open_stream(self) -> "Stream":
        return Stream(self)

    def counters(self) -> List[int]:
        out = (C.c_uint64 * 8)()
        _check(self.lib.dc_get_counters(self.handle, out), "dc_get_counters")
        return list(out)

    def profile_begin(self, max_launches: int = 1 << 16):
        _check(self.lib.dc_profile_begin(self.handle, max_launches), "dc_profile_begin")

    def profile_end(self):
        """Returns ({class: ms}, {class: launches}) summed since profile_begin."""
        ms = (C.c_double * 8)()
        n = (C.c_uint64 * 8)()
        _check(self.lib.dc_profile_end(self.handle, ms, n), "dc_profile_end")
        names = ["gemm_conv", "gemm_proj", "attention", "rmsnorm", "prep", "tapconv_f32", "head_istft_f32", "gemm_pair"]
        return ({k: ms[i] for i, k in enumerate(names)}, {k: n[i] for i, k in enumerate(names)})

    def destroy(self):
        if self.handle:
            _check(self.lib.dc_destroy(self.handle), "dc_destroy")
            self.handle = C.c_void_p()


class Stream:
    """dc_stream_open / dc_decode_chunk / dc_stream_reset / dc_stream_close."""

    def __init__(self, model: Model):
        self.model = model
        self.lib = model.lib
        self.handle = C.c_void_p()
        _check(self.lib.dc_stream_open(model.handle, C.byref(self.handle)), "dc_stream_open")

    def decode_chunk(self, feats, out=None, stream=None):
        """feats: CUDA float32 tensor [T, in_dim]; returns a CUDA float32 tensor."""
        import torch
        assert feats.is_cuda and feats.dtype == torch.float32 and feats.is_contiguous()
        T = feats.shape[0]
        if out is None:
            n = max(T, 0) * self.model.out_per_frame
            out = torch.empty(max(n, 1), dtype=torch.float32, device=feats.device)
        n_out = C.c_int(0)
        st = self.lib.dc_decode_chunk(self.handle, feats.data_ptr(), T, out.data_ptr(), C.byref(n_out),
                                      _cuda_stream_handle(stream))
        _check(st, "dc_decode_chunk")
        res = out[: n_out.value]
        if self.model.cfg.pipeline not in ("vocoder", "token2wav"):
            res = res.view(-1, self.model.out_per_frame)      # committed frames (fewer than T when the call carried look-ahead frames)
        return res

    def decode_wavefront(self, feats, out=None, stream=None):
        """dc_decode_wavefront: feats is a CUDA float32 tensor [n_frames, in_dim] holding all the stream's
        remaining input; returns what the chunk-by-chunk calls would have returned, concatenated."""
        import torch
        assert feats.is_cuda and feats.dtype == torch.float32 and feats.is_contiguous()
        n = feats.shape[0]
        if out is None:
            out = torch.empty(n * self.model.out_per_frame, device=feats.device, dtype=torch.float32)
        n_out = C.c_longlong(0)
        st = self.lib.dc_decode_wavefront(self.handle, feats.data_ptr(), n, out.data_ptr(), C.byref(n_out),
                                          _cuda_stream_handle(stream))
        _check(st, "dc_decode_wavefront")
        res = out[: n_out.value]
        if self.model.cfg.pipeline not in ("vocoder", "token2wav"):
            res = res.view(-1, self.model.out_per_frame)
        return res

    def decode_chunk_host(self, feats_host, out_host, stream=None) -> int:
        """feats_host / out_host: CPU float32 tensors (pinned for true async copies)."""
        T = feats_host.shape[0]
        n_out = C.c_int(0)
        st = self.lib.dc_decode_chunk_host(self.handle, feats_host.data_ptr(), T, out_host.data_ptr(),
                                           C.byref(n_out), _cuda_stream_handle(stream))
        _check(st, "dc_decode_chunk_host")
        return n_out.value

    def decode_raw(self, feats_ptr: int, T: int, out_ptr: int, stream=None) -> int:
        """Unchecked pass-through (used by the error-path tests)."""
        n_out = C.c_int(0)
        return self.lib.dc_decode_chunk(self.handle, feats_ptr, T, out_ptr, C.byref(n_out),
                                        _cuda_stream_handle(stream))

    def carry_info(self):
        buf = (C.c_uint64 * 256)()
        n = C.c_int(0)
        _check(self.lib.dc_stream_carry_info(self.handle, buf, 128, C.byref(n)), "dc_stream_carry_info")
        return [(buf[2 * i], buf[2 * i + 1]) for i in range(min(n.value, 128))]

    def snapshot(self, stream=None) -> "Snapshot":
        """Device-side copy of every carry of the stream plus its clocks (dc_stream_snapshot)."""
        h = C.c_void_p()
        _check(self.lib.dc_stream_snapshot(self.handle, C.byref(h), _cuda_stream_handle(stream)), "dc_stream_snapshot")
        return Snapshot(self.lib, h)

    def restore(self, snap: "Snapshot", stream=None):
        """Writes a snapshot back in place (of this stream or of another stream of the same model)."""
        _check(self.lib.dc_stream_restore(self.handle, snap.handle, _cuda_stream_handle(stream)), "dc_stream_restore")

    def check_guards(self) -> int:
        """dc_stream_check_guards: returns the number of damaged guard zones (0 = intact); raises on other errors."""
        n = C.c_int(0)
        st = self.lib.dc_stream_check_guards(self.handle, C.byref(n))
        if st not in (0, 7):
            _check(st, "dc_stream_check_guards")
        return n.value

    def reset(self, stream=None):
        _check(self.lib.dc_stream_reset(self.handle, _cuda_stream_handle(stream)), "dc_stream_reset")

    def close(self):
        if self.handle:
            _check(self.lib.dc_stream_close(self.handle), "dc_stream_close")
            self.handle = C.c_void_p()


def _ptr_array(items, n):
    """Pointers of n chunks: a list of tensors, or one contiguous tensor [n, T, width] (fast path)."""
    if hasattr(items, "data_ptr"):
        assert items.is_contiguous() and items.shape[0] == n
        stride = items.stride(0) * items.element_size()
        ptrs = items.data_ptr() + stride * np.arange(n, dtype=np.uint64)
        return (C.c_void_p * n).from_buffer_copy(ptrs.astype(np.uint64).tobytes()), items.shape[1]
    return (C.c_void_p * n)(*[t.data_ptr() for t in items]), None


def _batch_args(model: Model, streams: Sequence[Stream], feats, outs):
    n = len(streams)
    key = tuple(id(s) for s in streams)
    cache = model.__dict__.setdefault("_handle_cache", {})
    hs = cache.get(key)
    if hs is None:
        hs = cache[key] = (C.c_void_p * n)(*[s.handle for s in streams])
    fp, T = _ptr_array(feats, n)
    op, _ = _ptr_array(outs, n)
    nf = (C.c_int * n)(*([T] * n if T is not None else [f.shape[0] for f in feats]))
    return n, hs, fp, nf, op


def decode_batch_host(model: Model, streams: Sequence[Stream], feats_host, outs_host, stream=None):
    """dc_decode_batch_host: feats_host / outs_host are lists of CPU float32 tensors, or single contiguous
    CPU tensors [n_streams, T, width] (one chunk per stream)."""
    n, hs, fp, nf, op = _batch_args(model, streams, feats_host, outs_host)
    _check(model.lib.dc_decode_batch_host(model.handle, n, hs, fp, nf, op, _cuda_stream_handle(stream)),
           "dc_decode_batch_host")


def decode_batch(model: Model, streams: Sequence[Stream], feats, outs, stream=None):
    """dc_decode_batch: one chunk for each stream; feats / outs are lists of CUDA float32 tensors
    ([T_i, in_dim] / [T_i, out]) or single contiguous CUDA tensors [n_streams, T, width]."""
    n, hs, fp, nf, op = _batch_args(model, streams, feats, outs)
    _check(model.lib.dc_decode_batch(model.handle, n, hs, fp, nf, op, _cuda_stream_handle(stream)),
           "dc_decode_batch")


def decode_wavefront_batch(model: Model, streams: Sequence[Stream], feats, outs=None, stream=None):
    """dc_decode_wavefront_batch: feats[i] is a CUDA float32 tensor [n_frames_i, in_dim] with all of stream i's
    remaining input; returns the list of outputs (allocated here unless given)."""
    import torch
    n = len(streams)
    if outs is None:
        outs = [torch.empty(f.shape[0] * model.out_per_frame, device=f.device, dtype=torch.float32) for f in feats]
    for f in feats:
        assert f.is_cuda and f.dtype == torch.float32 and f.is_contiguous()
    hs = (C.c_void_p * n)(*[s.handle for s in streams])
    fp = (C.c_void_p * n)(*[f.data_ptr() for f in feats])
    nf = (C.c_longlong * n)(*[f.shape[0] for f in feats])
    op = (C.c_void_p * n)(*[o.data_ptr() for o in outs])
    _check(model.lib.dc_decode_wavefront_batch(model.handle, n, hs, fp, nf, op, _cuda_stream_handle(stream)),
           "dc_decode_wavefront_batch")
    if model.cfg.pipeline not in ("vocoder", "token2wav"):
        outs = [o.view(-1, model.out_per_frame) for o in outs]
    return outs


def measure_fp32_peak() -> float:
    """dc_measure_fp32_peak: measured FP32 multiply-add throughput of the current device in TFLOP/s."""
    v = C.c_double(0.0)
    _check(load_library().dc_measure_fp32_peak(C.byref(v)), "dc_measure_fp32_peak")
    return v.value


def fail_allocation(nth: int) -> None:
    """dc_test_fail_allocation: the nth device allocation of the calling thread from now on fails (0 disarms)."""
    _check(load_library().dc_test_fail_allocation(nth), "dc_test_fail_allocation")


def selftest_bounded_wait(max_polls: int = 1000) -> int:
    """dc_selftest_bounded_wait: returns the dc_status (6 = DC_ERR_TIMEOUT is the expected outcome)."""
    return load_library().dc_selftest_bounded_wait(max_polls)


NOALLOC_SCRATCH_FLOATS = 1 << 19


def conv_stack_noalloc(weights_dev, hidden: int, dilations: Sequence[int], x, y, stream=None) -> int:
    """dc_conv_stack_noalloc: the conv residual stack over one whole sequence, for callers that
    must not allocate device memory.  weights_dev, x, y are CUDA float32 tensors the caller owns;
    returns the dc_status (0 = DC_OK) so that refusals can be inspected."""
    lib = load_library()
    d = (C.c_int * len(dilations))(*dilations)
    return lib.dc_conv_stack_noalloc(weights_dev.data_ptr(), hidden, len(dilations), d, x.data_ptr(),
                                     x.shape[0], y.data_ptr(), _cuda_stream_handle(stream))
