"""Seeded synthetic workloads for the streaming decoder step.

This module serves both the CPU oracle and the CUDA path and therefore holds
none of the method's arithmetic: it only describes configurations (plain
data), enumerates the canonical weight blob (names, shapes, fan-in) and draws
Gaussian weights and inputs from ``numpy.random.default_rng(seed)`` in a fixed
order.  The decoder geometry follows the paper's streaming declaration
(Section 3.1: 50-frame chunks, 10 solver steps, retained history capped by the
retention policy); the layer widths come from the five benchmark
configurations.

Canonical weight blob (flat float32, this order)
------------------------------------------------
conv pipeline   per block:  W[3][C][C] (tap-major, tap 2 = current frame), b[C]
flow pipeline   W_in[2*mel][C], b_in[C];
                per group (conv_per_attn conv blocks then one attention layer):
                  per conv block: W[3][C][C], b[C], P[C][C]   (tau = emb @ P)
                  attention:      W_q, W_k, W_v, W_o [C][C], b_q, b_k, b_v, b_o [C]
                W_out[C][mel], b_out[mel]
vocoder         W_pre[3][mel][C0], b_pre[C0];
                per stage q: Wt[2*stride][C_in][C_out], bt[C_out],
                  per residual block: W[3][C_out][C_out], b[C_out]
                W_head[3][C3][n_fft+2], b_head[n_fft+2]
All matrices are input-major ([C_in][C_out]); a frame row vector multiplies
from the left.
"""
from __future__ import annotations

import dataclasses
import math
from dataclasses import dataclass, field
from typing import Dict, List, Tuple

import numpy as np

PIPE_CONV = "conv"
PIPE_FLOW = "flow"
PIPE_VOCODER = "vocoder"
PIPE_TOKEN2WAV = "token2wav"           # flow decoder feeding the vocoder tail inside one decode call


@dataclass(frozen=True)
class DCConfig:
    name: str
    pipeline: str                       # conv | flow | vocoder | token2wav
    precision: str                      # f32 | bf16 (fp32 accumulate)
    hidden: int = 0                     # C
    dilations: Tuple[int, ...] = ()     # one per conv block (flow / conv pipelines)
    n_attn_layers: int = 0
    n_heads: int = 0
    head_dim: int = 0
    kv_cap: int = 0                     # W, frames of carried keys/values (the retained history)
    f_prompt: int = 0                   # the stream's first f_prompt frames are a prompt that is never evicted
    f_lookahead: int = 0                # a full call of f_chunk frames also presents this many provisional frames
    n_steps: int = 0                    # Euler steps per chunk
    f_chunk: int = 50                   # admission bound on frames per call
    mel_dim: int = 80
    up_strides: Tuple[int, ...] = ()    # vocoder
    up_channels: Tuple[int, ...] = ()   # vocoder, len = len(up_strides)+1
    res_dilations: Tuple[int, ...] = (1, 2)
    n_fft: int = 16
    hop: int = 4
    rms_eps: float = 1e-6
    logmag_clamp: float = math.log(100.0)
    noise_seed: int = 0                 # flow decoder: != 0: the Euler noise x_0 is drawn on the device (Philox), feats = mu only
    cfg_scale: float = 0.0              # flow decoder: classifier-free guidance weight w (0 = off, one pass per step)
    excitation_std: float = 0.0         # vocoder: > 0: Gaussian excitation of this standard deviation, drawn on the device, added
    excitation_seed: int = 0            # ... after the last transposed conv (its generator key; must be != 0 then)
    # workload (not part of the network)
    n_chunks: int = 1
    n_streams: int = 1
    seed: int = 0
    bias_std: float = 0.0               # benchmark configs use zero biases

    @property
    def conv_per_attn(self) -> int:
        if self.n_attn_layers == 0:
            return len(self.dilations)
        assert len(self.dilations) % self.n_attn_layers == 0
        return len(self.dilations) // self.n_attn_layers

    @property
    def in_dim(self) -> int:
        """Width of one input frame handed to decode_chunk."""
        if self.pipeline == PIPE_CONV:
            return self.hidden
        if self.pipeline in (PIPE_FLOW, PIPE_TOKEN2WAV):
            if self.noise_seed:
                return self.mel_dim      # the conditioning mu; the noise x0 is drawn by the decoder itself
            return 2 * self.mel_dim      # cols [0,mel) = conditioning mu, [mel,2mel) = noise x0
        return self.mel_dim

    @property
    def out_per_frame(self) -> int:
        if self.pipeline == PIPE_CONV:
            return self.hidden
        if self.pipeline == PIPE_FLOW:
            return self.mel_dim
        up = 1
        for s in self.up_strides:
            up *= s
        return up * self.hop

    def replace(self, **kw) -> "DCConfig":
        return dataclasses.replace(self, **kw)

    # token2wav = the flow decoder (bf16) followed by the vocoder tail (fp32): the two halves as
    # configurations of their own (weights: the flow blob, then the vocoder blob)
    def flow_part(self) -> "DCConfig":
        assert self.pipeline == PIPE_TOKEN2WAV
        return self.replace(name=self.name + ".flow", pipeline=PIPE_FLOW, precision="bf16", excitation_std=0.0, excitation_seed=0)

    def vocoder_part(self) -> "DCConfig":
        assert self.pipeline == PIPE_TOKEN2WAV
        return self.replace(name=self.name + ".vocoder", pipeline=PIPE_VOCODER, precision="f32", noise_seed=0, cfg_scale=0.0,
                            f_prompt=0, f_lookahead=0)


def blob_layout(cfg: DCConfig) -> List[Tuple[str, Tuple[int, ...], int]]:
    """(name, shape, fan_in) of every tensor of the canonical blob, in order.
    fan_in == 0 marks a bias."""
    out: List[Tuple[str, Tuple[int, ...], int]] = []
    C = cfg.hidden
    if cfg.pipeline == PIPE_TOKEN2WAV:
        return blob_layout(cfg.flow_part()) + blob_layout(cfg.vocoder_part())
    if cfg.pipeline == PIPE_CONV:
        for l in range(len(cfg.dilations)):
            out.append((f"conv{l}.W", (3, C, C), 3 * C))
            out.append((f"conv{l}.b", (C,), 0))
    elif cfg.pipeline == PIPE_FLOW:
        m = cfg.mel_dim
        out.append(("in.W", (2 * m, C), 2 * m))
        out.append(("in.b", (C,), 0))
        cpa = cfg.conv_per_attn
        n_groups = max(cfg.n_attn_layers, 1)
        l = 0
        for g in range(n_groups):
            for _ in range(cpa):
                out.append((f"conv{l}.W", (3, C, C), 3 * C))
                out.append((f"conv{l}.b", (C,), 0))
                out.append((f"conv{l}.P", (C, C), C))
                l += 1
            if cfg.n_attn_layers:
                for nm in ("Wq", "Wk", "Wv", "Wo"):
                    out.append((f"attn{g}.{nm}", (C, C), C))
                for nm in ("bq", "bk", "bv", "bo"):
                    out.append((f"attn{g}.{nm}", (C,), 0))
        out.append(("out.W", (C, m), C))
        out.append(("out.b", (m,), 0))
    elif cfg.pipeline == PIPE_VOCODER:
        ch = cfg.up_channels
        out.append(("pre.W", (3, cfg.mel_dim, ch[0]), 3 * cfg.mel_dim))
        out.append(("pre.b", (ch[0],), 0))
        for q, s in enumerate(cfg.up_strides):
            ci, co = ch[q], ch[q + 1]
            out.append((f"up{q}.Wt", (2 * s, ci, co), 2 * ci))
            out.append((f"up{q}.bt", (co,), 0))
            for r in range(len(cfg.res_dilations)):
                out.append((f"up{q}.res{r}.W", (3, co, co), 3 * co))
                out.append((f"up{q}.res{r}.b", (co,), 0))
        nh = cfg.n_fft + 2
        out.append(("head.W", (3, ch[-1], nh), 3 * ch[-1]))
        out.append(("head.b", (nh,), 0))
    else:
        raise ValueError(cfg.pipeline)
    return out


def blob_size(cfg: DCConfig) -> int:
    return sum(int(np.prod(s)) for _, s, _ in blob_layout(cfg))


def make_weights(cfg: DCConfig, rng: np.random.Generator) -> np.ndarray:
    """Flat float32 blob: N(0, 1/fan_in) matrices, N(0, bias_std^2) biases."""
    parts = []
    for _, shape, fan_in in blob_layout(cfg):
        n = int(np.prod(shape))
        z = rng.standard_normal(n, dtype=np.float32)
        if fan_in:
            z *= np.float32(1.0 / math.sqrt(fan_in))
        else:
            z *= np.float32(cfg.bias_std)
        parts.append(z)
    return np.concatenate(parts).astype(np.float32)


@dataclass
class StreamInput:
    feats: np.ndarray                    # [F, in_dim] float32
    boundaries: List[int]                # 0 = B_0 < B_1 < ... < B_J = F


@dataclass
class Workload:
    cfg: DCConfig
    weights: np.ndarray                  # flat float32 blob
    streams: List[StreamInput] = field(default_factory=list)


def make_workload(cfg: DCConfig, boundaries: List[List[int]] | None = None) -> Workload:
    """Draw weights, then per stream: the chunk offset (multi-stream configs),
    then the whole stream's input frames.  `boundaries` overrides the chunk
    partition (one list per stream) for tests with ragged chunks."""
    rng = np.random.default_rng(cfg.seed)
    w = make_weights(cfg, rng)
    streams = []
    for i in range(cfg.n_streams):
        if boundaries is not None:
            b = list(boundaries[i])
        else:
            b = [0]
            if cfg.n_streams > 1:
                # first chunk of stream i has o_i frames (o_i drawn in [0, f_chunk)); o_i = 0
                # means an ordinary full first chunk
                o = int(rng.integers(0, cfg.f_chunk))
                if o > 0:
                    b.append(o)
            while len(b) - 1 < cfg.n_chunks:
                b.append(b[-1] + cfg.f_chunk)
        F = b[-1]
        feats = rng.standard_normal((F, cfg.in_dim), dtype=np.float32)
        streams.append(StreamInput(feats=feats, boundaries=b))
    return Workload(cfg=cfg, weights=w, streams=streams)


# --- the five benchmark configurations -------------------------------------------------------

CONFIGS: Dict[str, DCConfig] = {
    "cfg1": DCConfig(name="cfg1", pipeline=PIPE_CONV, precision="f32", hidden=64,
                     dilations=(1, 2), f_chunk=16, n_chunks=8, seed=0),
    "cfg2": DCConfig(name="cfg2", pipeline=PIPE_FLOW, precision="bf16", hidden=256,
                     dilations=(1, 1, 1, 1), n_attn_layers=2, n_heads=8, head_dim=32,
                     kv_cap=256, n_steps=10, f_chunk=50, n_chunks=40, seed=1),
    "cfg3": DCConfig(name="cfg3", pipeline=PIPE_FLOW, precision="bf16", hidden=512,
                     dilations=(1, 2, 4) * 4, n_attn_layers=4, n_heads=8, head_dim=64,
                     kv_cap=512, n_steps=10, f_chunk=50, n_chunks=100, seed=2),
    "cfg4": DCConfig(name="cfg4", pipeline=PIPE_VOCODER, precision="f32",
                     up_strides=(8, 5, 3), up_channels=(512, 256, 128, 64),
                     f_chunk=50, n_chunks=200, seed=3),
    "cfg5": DCConfig(name="cfg5", pipeline=PIPE_FLOW, precision="bf16", hidden=512,
                     dilations=(1, 2, 4) * 4, n_attn_layers=4, n_heads=8, head_dim=64,
                     kv_cap=512, n_steps=10, f_chunk=50, n_chunks=100, n_streams=32, seed=4),
}


def tiny_flow(**kw) -> DCConfig:
    """A small flow-decoder configuration for fast tests (same structure as cfg2)."""
    base = DCConfig(name="tiny_flow", pipeline=PIPE_FLOW, precision="bf16", hidden=64,
                    dilations=(1, 2), n_attn_layers=2, n_heads=2, head_dim=32, kv_cap=24,
                    n_steps=3, f_chunk=10, n_chunks=6, seed=11, bias_std=0.1)
    return base.replace(**kw)


def token2wav(**kw) -> DCConfig:
    """cfg3's flow decoder feeding cfg4's vocoder tail: one call turns a 50-frame chunk of
    [conditioning | noise] into 24,000 PCM samples (the whole decoder step of the method)."""
    f, v = CONFIGS["cfg3"], CONFIGS["cfg4"]
    base = f.replace(name="token2wav", pipeline=PIPE_TOKEN2WAV, up_strides=v.up_strides, up_channels=v.up_channels,
                     res_dilations=v.res_dilations, n_chunks=20, seed=6)
    return base.replace(**kw)


def tiny_token2wav(**kw) -> DCConfig:
    f = tiny_flow()
    base = f.replace(name="tiny_token2wav", pipeline=PIPE_TOKEN2WAV, mel_dim=16, up_strides=(3, 2), up_channels=(16, 8, 8),
                     seed=13)
    return base.replace(**kw)


# beyond the five: the whole decoder step in one call
EXTRA_CONFIGS: Dict[str, DCConfig] = {
    "token2wav": token2wav(),
    # ... for 32 concurrent streams (cfg5's serving shape with the vocoder tail behind every stream)
    "token2wav_serving": token2wav(name="token2wav_serving", n_streams=32, n_chunks=100, seed=10),
    # cfg3 with classifier-free guidance (two passes per Euler step, the form the paper measures its flow step in)
    "cfg3_guided": CONFIGS["cfg3"].replace(name="cfg3_guided", cfg_scale=0.7, seed=7),
    # cfg3's network with the paper's carry: a 302-frame prompt that is never evicted + 100 retained frames
    "cfg3_paper_carry": CONFIGS["cfg3"].replace(name="cfg3_paper_carry", f_prompt=302, kv_cap=100, seed=8),
    # ... and the 6 look-ahead frames of its 56-frame calls: the paper's whole declaration for this decoder
    "cfg3_paper": CONFIGS["cfg3"].replace(name="cfg3_paper", f_prompt=302, kv_cap=100, f_lookahead=6, seed=9),
}


def tiny_vocoder(**kw) -> DCConfig:
    base = DCConfig(name="tiny_vocoder", pipeline=PIPE_VOCODER, precision="f32", mel_dim=8,
                    up_strides=(3, 2), up_channels=(16, 8, 8), f_chunk=5, n_chunks=5, seed=12,
                    bias_std=0.1)
    return base.replace(**kw)
