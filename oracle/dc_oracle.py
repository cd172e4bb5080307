"""CPU oracle for the streaming decoder step.  TEST INFRASTRUCTURE ONLY.

Plain, slow, float64 numpy restatement of what the per-chunk decoder step
computes.  Only the tests, the smoke check and the benchmark's cpu-baseline /
reference legs may import this module; the product path (the CUDA library and
its Python binding) never does, and shares no code, table or constant with it.

Two independent formulations are given for every pipeline:

* ``*_offline``  - the plain definition: the causal network evaluated over the
  whole concatenated input, with the chunk boundaries known (they only matter
  for attention: every frame of a chunk sees its whole chunk plus at most W
  carried frames before the chunk start).
* ``*Stream``    - chunk-by-chunk evaluation with explicit carries that are
  updated by "concatenate, compute, keep the last rows" (the stock discipline
  the paper's Eq. 4 replaces by an in-place write), or, for the KV carry,
  optionally by an in-place ring (``carry="ring"``), whose equality with the
  concatenating form is the content of Eq. 4.

The paper (a runtime-systems paper) fixes the streaming semantics - carried
state per solver step and layer (Section 3.1, product clock "solver step x mel
frame"), retention capped after inference (Section 3.1, envelope vs attended
extent), in-place carry (Section 3.2, Eq. 4), admission f <= f_chunk - but not
the layer arithmetic, which is fixed by the benchmark configurations and the
readings listed in the design notes.  Pins: see tests/test_oracle_*.py.
Whole-configuration outputs have no value printed in the paper: parity
unpinned against the paper for those; they are pinned by closed forms, brute
force, library special cases and the streamed == offline invariant.

Precision: all arithmetic in float64.  For ``precision == "bf16"`` the values
are additionally rounded (round-to-nearest-even to 8 significant bits) at the
declared storage points: weight matrices, the input-projection operand
[x_s | mu], every stored residual-stream activation h, the normalised
activation u, q, k, v, the unnormalised softmax numerators (the row sum uses
the unrounded ones) and the attention output o.  Biases, the timestep bias
tau, the Euler state x_s and all accumulations stay unrounded.
"""
from __future__ import annotations

import math
from typing import Tuple, Dict, List, Optional, Sequence

import numpy as np


# --------------------------------------------------------------------------------------------
# scalar helpers
# --------------------------------------------------------------------------------------------

def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round float64 values to the nearest bfloat16 (8-bit significand, ties to
    even), returned as float64.  Exponent range is not clamped (values here
    are O(1))."""
    x = np.asarray(x, dtype=np.float64)
    m, e = np.frexp(x)                       # x = m * 2**e, 0.5 <= |m| < 1
    return np.ldexp(np.rint(m * 256.0), e - 8)


def silu(z: np.ndarray) -> np.ndarray:
    return z / (1.0 + np.exp(-z))


def rmsnorm(h: np.ndarray, eps: float) -> np.ndarray:
    """Parameter-free RMS normalisation over the channel axis."""
    return h / np.sqrt(np.mean(h * h, axis=-1, keepdims=True) + eps)


def timestep_embedding(t: float, C: int) -> np.ndarray:
    """emb[i] = sin(1000 t w_i), emb[C/2+i] = cos(1000 t w_i), w_i = 10000^(-i/(C/2))."""
    half = C // 2
    i = np.arange(half, dtype=np.float64)
    w = 10000.0 ** (-i / half)
    return np.concatenate([np.sin(1000.0 * t * w), np.cos(1000.0 * t * w)])


def shift_rows(x: np.ndarray, delta: int, left: Optional[np.ndarray] = None) -> np.ndarray:
    """Row i of the result is row i-delta of x; rows before the start come from
    `left` (its last rows) or are zero."""
    F = x.shape[0]
    if left is None:
        left = np.zeros((delta, x.shape[1]))
    ext = np.concatenate([left[left.shape[0] - delta:], x], axis=0) if delta else x
    return ext[:F]


def causal_conv_k3(x: np.ndarray, W: np.ndarray, d: int,
                   left: Optional[np.ndarray] = None) -> np.ndarray:
    """y[i] = sum_{j=0..2} x[i-(2-j)d] @ W[j]  (cross-correlation, tap 2 = current
    frame); frames before the start are `left` (shape [2d, C_in]) or zeros."""
    if left is None:
        left = np.zeros((2 * d, x.shape[1]))
    y = np.zeros((x.shape[0], W.shape[2]))
    for j in range(3):
        y += shift_rows(x, (2 - j) * d, left) @ W[j]
    return y


# --------------------------------------------------------------------------------------------
# weights
# --------------------------------------------------------------------------------------------

def parse_blob(cfg, blob: np.ndarray) -> Dict[str, np.ndarray]:
    """Split the canonical flat float32 blob into named float64 tensors.  In bf16
    precision the matrices are rounded to bf16; biases are not."""
    blob = np.asarray(blob, dtype=np.float32)
    W: Dict[str, np.ndarray] = {}
    pos = 0
    bf = cfg.precision == "bf16"

    def take(name, shape, is_bias=False):
        nonlocal pos
        n = int(np.prod(shape))
        a = blob[pos:pos + n].astype(np.float64).reshape(shape)
        pos += n
        W[name] = round_bf16(a) if (bf and not is_bias) else a

    C = cfg.hidden
    if cfg.pipeline == "conv":
        for l in range(len(cfg.dilations)):
            take(f"conv{l}.W", (3, C, C))
            take(f"conv{l}.b", (C,), True)
    elif cfg.pipeline == "flow":
        m = cfg.mel_dim
        take("in.W", (2 * m, C))
        take("in.b", (C,), True)
        l = 0
        for g in range(max(cfg.n_attn_layers, 1)):
            for _ in range(cfg.conv_per_attn):
                take(f"conv{l}.W", (3, C, C))
                take(f"conv{l}.b", (C,), True)
                take(f"conv{l}.P", (C, C))
                l += 1
            if cfg.n_attn_layers:
                for nm in ("Wq", "Wk", "Wv", "Wo"):
                    take(f"attn{g}.{nm}", (C, C))
                for nm in ("bq", "bk", "bv", "bo"):
                    take(f"attn{g}.{nm}", (C,), True)
        take("out.W", (C, m))
        take("out.b", (m,), True)
    elif cfg.pipeline == "vocoder":
        ch = cfg.up_channels
        take("pre.W", (3, cfg.mel_dim, ch[0]))
        take("pre.b", (ch[0],), True)
        for q, s in enumerate(cfg.up_strides):
            take(f"up{q}.Wt", (2 * s, ch[q], ch[q + 1]))
            take(f"up{q}.bt", (ch[q + 1],), True)
            for r in range(len(cfg.res_dilations)):
                take(f"up{q}.res{r}.W", (3, ch[q + 1], ch[q + 1]))
                take(f"up{q}.res{r}.b", (ch[q + 1],), True)
        take("head.W", (3, ch[-1], cfg.n_fft + 2))
        take("head.b", (cfg.n_fft + 2,), True)
    else:
        raise ValueError(cfg.pipeline)
    if pos != blob.size:
        raise ValueError(f"weight blob has {blob.size} floats, layout needs {pos}")
    return W


def tau_table(cfg, W) -> np.ndarray:
    """tau[s][l] = emb(s / n_steps) @ P_l : the per-step, per-block timestep bias."""
    n, L, C = cfg.n_steps, len(cfg.dilations), cfg.hidden
    tau = np.zeros((n, L, C))
    for s in range(n):
        e = timestep_embedding(s / n, C)
        for l in range(L):
            tau[s, l] = e @ W[f"conv{l}.P"]
    return tau


# --------------------------------------------------------------------------------------------
# conv stack (tiny causal conv stream)
# --------------------------------------------------------------------------------------------

def conv_stack_offline(cfg, blob, x: np.ndarray) -> np.ndarray:
    """y = block_L(...block_1(x)),  block: h <- h + SiLU(conv_k3,d(h) + b)."""
    W = parse_blob(cfg, blob)
    h = np.asarray(x, dtype=np.float64)
    for l, d in enumerate(cfg.dilations):
        h = h + silu(causal_conv_k3(h, W[f"conv{l}.W"], d) + W[f"conv{l}.b"])
    return h.astype(np.float32)


class ConvStackStream:
    """Chunk-by-chunk conv stack; carry per block = last 2d input frames."""

    def __init__(self, cfg, blob):
        self.cfg = cfg
        self.W = parse_blob(cfg, blob)
        self.carry = [np.zeros((2 * d, cfg.hidden)) for d in cfg.dilations]

    def decode_chunk(self, x: np.ndarray) -> np.ndarray:
        h = np.asarray(x, dtype=np.float64)
        assert 1 <= h.shape[0] <= self.cfg.f_chunk
        for l, d in enumerate(self.cfg.dilations):
            left = self.carry[l]
            self.carry[l] = np.concatenate([left, h], axis=0)[-2 * d:]
            h = h + silu(causal_conv_k3(h, self.W[f"conv{l}.W"], d, left) + self.W[f"conv{l}.b"])
        return h.astype(np.float32)


# --------------------------------------------------------------------------------------------
# flow decoder
# --------------------------------------------------------------------------------------------

def _attend(cfg, q, k, v, rb):
    """All rows of q attend to all rows of k/v (one chunk against its key set).
    Per head: e = exp(s - max s), o = (rb(e) @ v) / sum(e)."""
    H, dh = cfg.n_heads, cfg.head_dim
    o = np.zeros_like(q)
    for eta in range(H):
        sl = slice(eta * dh, (eta + 1) * dh)
        s = (q[:, sl] @ k[:, sl].T) / math.sqrt(dh)
        e = np.exp(s - s.max(axis=1, keepdims=True))
        o[:, sl] = (rb(e) @ v[:, sl]) / e.sum(axis=1, keepdims=True)
    return rb(o)


def _layer_plan(cfg):
    """[('conv', l, d) ... ('attn', g)] in execution order."""
    plan, l = [], 0
    for g in range(max(cfg.n_attn_layers, 1)):
        for _ in range(cfg.conv_per_attn):
            plan.append(("conv", l, cfg.dilations[l]))
            l += 1
        if cfg.n_attn_layers:
            plan.append(("attn", g, 0))
    return plan


_PHILOX_M0, _PHILOX_M1 = np.uint64(0xD2511F53), np.uint64(0xCD9E8D57)
_PHILOX_W0, _PHILOX_W1 = 0x9E3779B9, 0xBB67AE85


def philox4x32_10(ctr: np.ndarray, key: Tuple[int, int]) -> np.ndarray:
    """Philox4x32 with 10 rounds (Salmon et al., "Parallel random numbers: as easy as 1, 2, 3", 2011),
    the counter-based generator of device random streams.  ctr: [..., 4] uint32 counters; returns the
    [..., 4] uint32 outputs."""
    c = [np.asarray(ctr[..., i], dtype=np.uint64) for i in range(4)]
    k0, k1 = int(key[0]) & 0xFFFFFFFF, int(key[1]) & 0xFFFFFFFF
    mask, sh = np.uint64(0xFFFFFFFF), np.uint64(32)
    for _ in range(10):
        p0, p1 = _PHILOX_M0 * c[0], _PHILOX_M1 * c[2]
        c = [(p1 >> sh) ^ c[1] ^ np.uint64(k0), p1 & mask, (p0 >> sh) ^ c[3] ^ np.uint64(k1), p0 & mask]
        k0, k1 = (k0 + _PHILOX_W0) & 0xFFFFFFFF, (k1 + _PHILOX_W1) & 0xFFFFFFFF
    return np.stack(c, axis=-1).astype(np.uint32)


def device_noise(seed: int, stream_id: int, frame0: int, n_frames: int, mel: int) -> np.ndarray:
    """The Euler noise x_0 of frames frame0 .. frame0 + n_frames - 1 when the decoder draws it itself:
    the draw of (frame t, channels 4g .. 4g+3) is Philox4x32-10 at counter (t mod 2^32, t div 2^32, g,
    stream id) under the key (seed mod 2^32, seed div 2^32) - the generator's offset is the stream's frame
    clock (Sec. 3.3, effect classification) - turned into four standard normals by two Box-Muller
    pairs on u = ((r >> 8) + 1/2) 2^-24."""
    t = np.arange(frame0, frame0 + n_frames, dtype=np.int64)[:, None]
    g = np.arange(mel // 4, dtype=np.int64)[None, :]
    ctr = np.stack(np.broadcast_arrays(t & 0xFFFFFFFF, t >> 32, g, np.int64(stream_id)), axis=-1).astype(np.uint32)
    r = philox4x32_10(ctr, (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)).astype(np.float64)
    u = (np.floor(r / 256.0) + 0.5) / 16777216.0
    rad0, rad1 = np.sqrt(-2.0 * np.log(u[..., 0])), np.sqrt(-2.0 * np.log(u[..., 2]))
    a0, a1 = 2.0 * np.pi * u[..., 1], 2.0 * np.pi * u[..., 3]
    z = np.stack([rad0 * np.cos(a0), rad0 * np.sin(a0), rad1 * np.cos(a1), rad1 * np.sin(a1)], axis=-1)
    return z.reshape(n_frames, mel)


def excitation_noise(seed: int, stream_id: int, t0: int, n: int, C: int) -> np.ndarray:
    """The vocoder's random excitation (the device-random source of Sec. 3.1 / Sec. 3.3 effect classification,
    clause (iii): admitted because its generator offset is a function of the call clock).  Rows are frames
    t0 .. t0 + n - 1 at the rate of the last upsampling stage, counted from the stream start; the draw of
    (frame t, channels 4g .. 4g+3) is Philox4x32-10 at counter (t mod 2^32, t div 2^32, g, 2^31 + stream id) -
    the high bit keeps these draws apart from the flow decoder's noise under the same key - under the key
    (seed mod 2^32, seed div 2^32), turned into four standard normals exactly as in device_noise."""
    t = np.arange(t0, t0 + n, dtype=np.int64)[:, None]
    g = np.arange(C // 4, dtype=np.int64)[None, :]
    ctr = np.stack(np.broadcast_arrays(t & 0xFFFFFFFF, t >> 32, g, np.int64((1 << 31) + stream_id)), axis=-1).astype(np.uint32)
    r = philox4x32_10(ctr, (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)).astype(np.float64)
    u = (np.floor(r / 256.0) + 0.5) / 16777216.0
    rad0, rad1 = np.sqrt(-2.0 * np.log(u[..., 0])), np.sqrt(-2.0 * np.log(u[..., 2]))
    a0, a1 = 2.0 * np.pi * u[..., 1], 2.0 * np.pi * u[..., 3]
    z = np.stack([rad0 * np.cos(a0), rad0 * np.sin(a0), rad1 * np.cos(a1), rad1 * np.sin(a1)], axis=-1)
    return z.reshape(n, C)


def attended_frames(cfg, lo: int, hi: int) -> np.ndarray:
    """Frames whose keys/values the chunk [lo, hi) attends (Sec. 3.1 "Two extents", Eq. 4): the
    prompt - the stream's first f_prompt frames, never evicted - then the last <= kv_cap frames of
    history after the prompt, then the chunk itself.  f_prompt = 0: a plain sliding window."""
    P = getattr(cfg, "f_prompt", 0)
    prompt = np.arange(0, min(P, hi))                                   # including the prompt frames this chunk brings
    history = np.arange(max(P, lo - cfg.kv_cap), lo) if lo > P else np.arange(0)   # last <= kv_cap frames after the prompt
    own = np.arange(max(lo, P), hi)
    return np.concatenate([prompt, history, own]).astype(np.int64)


def flow_offline(cfg, blob, feats: np.ndarray, boundaries: Sequence[int], stream_id: int = 0) -> np.ndarray:
    """Offline causal run over the concatenated input.  feats[:, :mel] is the
    conditioning mu, feats[:, mel:] the initial noise x_0.  For s in 0..n-1:
    h = [x_s | mu] W_in + b_in; conv blocks h <- h + SiLU(conv(h) + b + tau_{s,l});
    attention h <- h + attn(rmsnorm(h)) W_o + b_o with keys
    K(i) = { j : max(0, B_c(i) - W) <= j < B_{c(i)+1} };
    v = rmsnorm(h) W_out + b_out;  x_{s+1} = x_s + v / n.  Output x_n."""
    W = parse_blob(cfg, blob)
    rb = round_bf16 if cfg.precision == "bf16" else (lambda a: a)
    m, n = cfg.mel_dim, cfg.n_steps
    feats = np.asarray(feats, dtype=np.float64)
    F = feats.shape[0]
    if getattr(cfg, "noise_seed", 0):
        mu, x = feats, device_noise(cfg.noise_seed, stream_id, 0, F, m)
    else:
        mu, x = feats[:, :m], feats[:, m:].copy()
    assert boundaries[0] == 0 and boundaries[-1] == F
    tau = tau_table(cfg, W)
    plan = _layer_plan(cfg)

    def velocity(s, x, cond):
        h = rb(rb(np.concatenate([x, cond], axis=1)) @ W["in.W"] + W["in.b"])
        for kind, idx, d in plan:
            if kind == "conv":
                z = causal_conv_k3(h, W[f"conv{idx}.W"], d) + W[f"conv{idx}.b"] + tau[s, idx]
                h = rb(h + silu(z))
            else:
                u = rb(rmsnorm(h, cfg.rms_eps))
                q = rb(u @ W[f"attn{idx}.Wq"] + W[f"attn{idx}.bq"])
                k = rb(u @ W[f"attn{idx}.Wk"] + W[f"attn{idx}.bk"])
                v = rb(u @ W[f"attn{idx}.Wv"] + W[f"attn{idx}.bv"])
                o = np.zeros_like(q)
                for c in range(len(boundaries) - 1):
                    lo, hi = boundaries[c], boundaries[c + 1]
                    keys = attended_frames(cfg, lo, hi)
                    o[lo:hi] = _attend(cfg, q[lo:hi], k[keys], v[keys], rb)
                h = rb(h + o @ W[f"attn{idx}.Wo"] + W[f"attn{idx}.bo"])
        return rb(rmsnorm(h, cfg.rms_eps)) @ W["out.W"] + W["out.b"]

    w_cfg = getattr(cfg, "cfg_scale", 0.0)
    for s in range(n):
        vel = velocity(s, x, mu)
        if w_cfg > 0:
            # classifier-free guidance (the flow step of Table 1 is the guided one, batch x 2): a second pass
            # with the conditioning removed, v = (1 + w) v_cond - w v_uncond
            vel = (1.0 + w_cfg) * vel - w_cfg * velocity(s, x, np.zeros_like(mu))
        x = x + vel / n
    return x.astype(np.float32)


class KVRing:
    """In-place KV carry: fixed storage of W + f_chunk rows, written at the head;
    the attended rows are the last min(filled, W) + T rows ending at the head
    (Eq. 4's discipline: same values as concatenate-then-truncate, constant
    storage)."""

    def __init__(self, cap: int, f_call: int, C: int):
        self.cap, self.size = cap, cap + f_call
        self.k = np.zeros((self.size, C))
        self.v = np.zeros((self.size, C))
        self.head = 0          # next row to write
        self.filled = 0        # carried rows (<= cap)

    def append_and_view(self, k, v, n_commit: Optional[int] = None):
        """Writes the T rows at the head and returns the attended rows; the head only advances by
        n_commit rows (the others are look-ahead: attended now, overwritten by the next call)."""
        T = k.shape[0]
        nc = T if n_commit is None else n_commit
        idx = (self.head + np.arange(T, dtype=np.int64)) % self.size
        self.k[idx], self.v[idx] = k, v
        L = self.filled + T
        rows = (self.head + T - L + np.arange(L, dtype=np.int64)) % self.size
        self.head = (self.head + nc) % self.size
        self.filled = min(self.cap, self.filled + nc)
        return self.k[rows], self.v[rows]


class ConcatCarry:
    """The stock discipline of Eq. 4's right-hand side: the live cache H is a fresh concatenation,
    mutable history first (newest frame first: "prepend ordering"), immutable prompt tail last;
    the carry keeps H[0:kv_cap] and the prompt tail.  The stream's first f_prompt frames are the
    prompt."""

    def __init__(self, cap: int, f_prompt: int, C: int):
        self.cap, self.P = cap, f_prompt
        self.hist_k, self.hist_v = np.zeros((0, C)), np.zeros((0, C))
        self.prompt_k, self.prompt_v = np.zeros((0, C)), np.zeros((0, C))

    @property
    def filled(self) -> int:
        return self.hist_k.shape[0] + self.prompt_k.shape[0]

    def append_and_view(self, k, v, a0: int, n_commit: Optional[int] = None):
        """k, v: the call's frames (absolute index a0 ..); only the first n_commit are kept afterwards
        (look-ahead frames sit in the live cache H but are dropped before truncation)."""
        T = k.shape[0]
        nc = T if n_commit is None else n_commit
        tp = min(max(self.P - a0, 0), T)                    # call frames that are prompt frames
        live_prompt_k = np.concatenate([self.prompt_k, k[:tp]], axis=0)
        live_prompt_v = np.concatenate([self.prompt_v, v[:tp]], axis=0)
        live_k = np.concatenate([k[tp:][::-1], self.hist_k], axis=0)
        live_v = np.concatenate([v[tp:][::-1], self.hist_v], axis=0)
        H_k = np.concatenate([live_k, live_prompt_k], axis=0)
        H_v = np.concatenate([live_v, live_prompt_v], axis=0)
        # retention, after the inference that reads H: drop the look-ahead frames, then truncate
        tpc = min(tp, nc)
        self.prompt_k = np.concatenate([self.prompt_k, k[:tpc]], axis=0)
        self.prompt_v = np.concatenate([self.prompt_v, v[:tpc]], axis=0)
        drop = (T - tp) - max(nc - tp, 0)                   # look-ahead frames among the history frames (newest first)
        self.hist_k, self.hist_v = live_k[drop:][:self.cap], live_v[drop:][:self.cap]
        return H_k, H_v


class RingCarry:
    """The in-place discipline (Eq. 4's left-hand side): a prompt buffer of f_prompt rows written
    once, and a ring of kv_cap + f_chunk rows for the history; nothing is allocated per chunk."""

    def __init__(self, cap: int, f_chunk: int, f_prompt: int, C: int):
        self.P = f_prompt
        self.pk, self.pv = np.zeros((f_prompt, C)), np.zeros((f_prompt, C))
        self.n_prompt = 0
        self.ring = KVRing(cap, f_chunk, C)

    @property
    def filled(self) -> int:
        return self.n_prompt + self.ring.filled

    def append_and_view(self, k, v, a0: int, n_commit: Optional[int] = None):
        T = k.shape[0]
        nc = T if n_commit is None else n_commit
        tp = min(max(self.P - a0, 0), T)
        self.pk[self.n_prompt:self.n_prompt + tp], self.pv[self.n_prompt:self.n_prompt + tp] = k[:tp], v[:tp]
        n_live = self.n_prompt + tp                        # look-ahead rows are written too; the next call overwrites them
        self.n_prompt += min(tp, nc)
        hk, hv = self.ring.append_and_view(k[tp:], v[tp:], max(nc - tp, 0))
        return (np.concatenate([self.pk[:n_live], hk], axis=0),
                np.concatenate([self.pv[:n_live], hv], axis=0))


class FlowStream:
    """Chunk-by-chunk flow decoder.  State per Euler step s: per conv block the
    last 2d block-input frames; per attention layer the keys/values of the last
    <= W frames (empty at stream start)."""

    def __init__(self, cfg, blob, carry: str = "concat", stream_id: int = 0):
        self.cfg = cfg
        self.stream_id = stream_id            # selects the stream's device random stream (noise_seed != 0)
        self.W = parse_blob(cfg, blob)
        self.tau = tau_table(cfg, self.W)
        self.plan = _layer_plan(cfg)
        self.ring = carry == "ring"
        C, n = cfg.hidden, cfg.n_steps
        self.w_cfg = getattr(cfg, "cfg_scale", 0.0)
        # with classifier-free guidance the conditional and the unconditional pass each carry a state of their own
        self.passes = []
        for _ in range(2 if self.w_cfg > 0 else 1):
            halo = [[np.zeros((2 * d, C)) for d in cfg.dilations] for _ in range(n)]
            P = getattr(cfg, "f_prompt", 0)
            if self.ring:
                kv = [[RingCarry(cfg.kv_cap, cfg.f_chunk + getattr(cfg, "f_lookahead", 0), P, C)
                       for _ in range(cfg.n_attn_layers)] for _ in range(n)]
            else:
                kv = [[ConcatCarry(cfg.kv_cap, P, C) for _ in range(cfg.n_attn_layers)] for _ in range(n)]
            self.passes.append((halo, kv))
        self.halo, self.kv = self.passes[0]
        self.frames = 0                      # frames decoded so far = index of the next chunk's first frame
        self.kv_len_seen: List[int] = []

    def decode_chunk(self, feats: np.ndarray) -> np.ndarray:
        cfg, W = self.cfg, self.W
        rb = round_bf16 if cfg.precision == "bf16" else (lambda a: a)
        feats = np.asarray(feats, dtype=np.float64)
        T = feats.shape[0]
        la = getattr(cfg, "f_lookahead", 0)
        assert 1 <= T <= cfg.f_chunk + la
        # Frames beyond f_chunk are look-ahead (Sec. 3.1 "Two extents": they reside in the envelope, are attended
        # by the call, and are discarded before the retention policy truncates): the call commits the first Tc
        # frames - output, conv left context and K/V carry - and the caller presents the others again.
        self.Tc = min(T, cfg.f_chunk)
        m, n = cfg.mel_dim, cfg.n_steps
        if getattr(cfg, "noise_seed", 0):
            mu, x = feats, device_noise(cfg.noise_seed, self.stream_id, self.frames, T, m)   # look-ahead frames draw again next call
        else:
            mu, x = feats[:, :m], feats[:, m:].copy()
        for s in range(n):
            vel = self._velocity(s, x, mu, 0, rb)
            if self.w_cfg > 0:
                vel = (1.0 + self.w_cfg) * vel - self.w_cfg * self._velocity(s, x, np.zeros_like(mu), 1, rb)
            x = x + vel / n
        self.frames += self.Tc
        return x[:self.Tc].astype(np.float32)

    def _velocity(self, s, x, cond, p, rb):
        """One evaluation of the network at Euler step s with pass p's carries (updated in passing)."""
        cfg, W = self.cfg, self.W
        halo, kv = self.passes[p]
        h = rb(rb(np.concatenate([x, cond], axis=1)) @ W["in.W"] + W["in.b"])
        for kind, idx, d in self.plan:
            if kind == "conv":
                left = halo[s][idx]
                halo[s][idx] = np.concatenate([left, h[:self.Tc]], axis=0)[-2 * d:]
                z = (causal_conv_k3(h, W[f"conv{idx}.W"], d, left)
                     + W[f"conv{idx}.b"] + self.tau[s, idx])
                h = rb(h + silu(z))
            else:
                u = rb(rmsnorm(h, cfg.rms_eps))
                q = rb(u @ W[f"attn{idx}.Wq"] + W[f"attn{idx}.bq"])
                k = rb(u @ W[f"attn{idx}.Wk"] + W[f"attn{idx}.bk"])
                v = rb(u @ W[f"attn{idx}.Wv"] + W[f"attn{idx}.bv"])
                if s == 0 and idx == 0 and p == 0:
                    self.kv_len_seen.append(kv[s][idx].filled)
                k_all, v_all = kv[s][idx].append_and_view(k, v, self.frames, self.Tc)
                o = _attend(cfg, q, k_all, v_all, rb)
                h = rb(h + o @ W[f"attn{idx}.Wo"] + W[f"attn{idx}.bo"])
        return rb(rmsnorm(h, cfg.rms_eps)) @ W["out.W"] + W["out.b"]


# --------------------------------------------------------------------------------------------
# vocoder tail: upsampler + head + iSTFT / overlap-add
# --------------------------------------------------------------------------------------------

def conv_transpose_causal(x: np.ndarray, Wt: np.ndarray, b: np.ndarray, stride: int,
                          prev: Optional[np.ndarray] = None) -> np.ndarray:
    """y[stride*n + r] = b + x[n] @ Wt[r] + x[n-1] @ Wt[r+stride], r in [0, stride);
    x[-1] = prev (zeros at stream start).  This is ConvTranspose1d(stride, kernel
    2*stride) with the trailing `stride` outputs deferred to the next frame."""
    F = x.shape[0]
    if prev is None:
        prev = np.zeros((1, x.shape[1]))
    xm1 = np.concatenate([prev.reshape(1, -1), x], axis=0)[:F]
    y = np.zeros((F, stride, Wt.shape[2]))
    for r in range(stride):
        y[:, r, :] = b + x @ Wt[r] + xm1 @ Wt[r + stride]
    return y.reshape(F * stride, Wt.shape[2])


def hann_periodic(N: int) -> np.ndarray:
    return 0.5 - 0.5 * np.cos(2.0 * np.pi * np.arange(N) / N)


def frame_signal(z: np.ndarray, n_fft: int, clamp: float) -> np.ndarray:
    """Head output z [M, n_fft+2] -> per-frame real signal xi [M, n_fft].
    Channels [0, n_fft/2] are log-magnitudes (clamped from above), the rest are
    phases; X_f = exp(m_f)(cos phi_f + i sin phi_f); inverse real DFT with 1/N
    scaling, imaginary parts of the DC and Nyquist bins ignored."""
    nb = n_fft // 2 + 1
    mag = np.exp(np.minimum(z[:, :nb], clamp))
    re, im = mag * np.cos(z[:, nb:]), mag * np.sin(z[:, nb:])
    kap = np.arange(n_fft)
    xi = re[:, 0:1] + re[:, nb - 1:nb] * ((-1.0) ** kap)[None, :]
    for f in range(1, nb - 1):
        ang = 2.0 * np.pi * f * kap / n_fft
        xi = xi + 2.0 * (re[:, f:f + 1] * np.cos(ang)[None, :] - im[:, f:f + 1] * np.sin(ang)[None, :])
    return xi / n_fft


def ola_norm(n_fft: int, hop: int) -> float:
    """Steady-state overlap-add envelope sum_j w[j*hop]^2 (1.5 for periodic Hann, hop N/4)."""
    w = hann_periodic(n_fft)
    return float(sum(w[j] ** 2 for j in range(0, n_fft, hop)))


def overlap_add(xi: np.ndarray, n_fft: int, hop: int, tail: Optional[np.ndarray] = None):
    """pcm[n] = (1/norm) sum_m w[n - hop m] xi_m[n - hop m]; returns the hop*M
    finalised samples and the (n_fft - hop)-sample unnormalised tail to carry."""
    M = xi.shape[0]
    w = hann_periodic(n_fft)
    acc = np.zeros(hop * M + n_fft - hop)
    if tail is not None:
        acc[:n_fft - hop] += tail
    for mfr in range(M):
        acc[hop * mfr: hop * mfr + n_fft] += w * xi[mfr]
    return acc[:hop * M] / ola_norm(n_fft, hop), acc[hop * M:]


def vocoder_offline(cfg, blob, mel: np.ndarray, stream_id: int = 0) -> np.ndarray:
    """The vocoder tail over a whole sequence.  With cfg.excitation_std > 0 the output of the LAST transposed
    conv (before that stage's residual blocks) receives excitation_std * excitation_noise."""
    W = parse_blob(cfg, blob)
    a = causal_conv_k3(np.asarray(mel, dtype=np.float64), W["pre.W"], 1) + W["pre.b"]
    for q, s in enumerate(cfg.up_strides):
        a = conv_transpose_causal(a, W[f"up{q}.Wt"], W[f"up{q}.bt"], s)
        if q == len(cfg.up_strides) - 1 and getattr(cfg, "excitation_std", 0.0) > 0.0:
            a = a + cfg.excitation_std * excitation_noise(cfg.excitation_seed, stream_id, 0, a.shape[0], a.shape[1])
        for r, d in enumerate(cfg.res_dilations):
            a = a + silu(causal_conv_k3(a, W[f"up{q}.res{r}.W"], d) + W[f"up{q}.res{r}.b"])
    z = causal_conv_k3(silu(a), W["head.W"], 1) + W["head.b"]
    xi = frame_signal(z, cfg.n_fft, cfg.logmag_clamp)
    pcm, _ = overlap_add(xi, cfg.n_fft, cfg.hop)
    return pcm.astype(np.float32)


class VocoderStream:
    """Chunk-by-chunk vocoder tail.  Carries: last 2 mel frames, last input frame
    of each transposed conv, last 2d input frames of each residual block, last 2
    frames before the head, and the n_fft - hop overlap-add partial sums."""

    def __init__(self, cfg, blob, stream_id: int = 0):
        self.cfg = cfg
        self.W = parse_blob(cfg, blob)
        self.stream_id = stream_id
        self.t_exc = 0                 # frames emitted so far at the last stage's rate: the excitation's clock
        ch = cfg.up_channels
        self.c_pre = np.zeros((2, cfg.mel_dim))
        self.c_up = [np.zeros((1, ch[q])) for q in range(len(cfg.up_strides))]
        self.c_res = [[np.zeros((2 * d, ch[q + 1])) for d in cfg.res_dilations]
                      for q in range(len(cfg.up_strides))]
        self.c_head = np.zeros((2, ch[-1]))
        self.tail = np.zeros(cfg.n_fft - cfg.hop)

    def decode_chunk(self, mel: np.ndarray) -> np.ndarray:
        cfg, W = self.cfg, self.W
        x = np.asarray(mel, dtype=np.float64)
        assert 1 <= x.shape[0] <= cfg.f_chunk
        left, self.c_pre = self.c_pre, np.concatenate([self.c_pre, x], axis=0)[-2:]
        a = causal_conv_k3(x, W["pre.W"], 1, left) + W["pre.b"]
        for q, s in enumerate(cfg.up_strides):
            prev, self.c_up[q] = self.c_up[q], a[-1:].copy()
            a = conv_transpose_causal(a, W[f"up{q}.Wt"], W[f"up{q}.bt"], s, prev)
            if q == len(cfg.up_strides) - 1 and getattr(cfg, "excitation_std", 0.0) > 0.0:
                a = a + cfg.excitation_std * excitation_noise(cfg.excitation_seed, self.stream_id, self.t_exc, a.shape[0], a.shape[1])
                self.t_exc += a.shape[0]
            for r, d in enumerate(cfg.res_dilations):
                left = self.c_res[q][r]
                self.c_res[q][r] = np.concatenate([left, a], axis=0)[-2 * d:]
                a = a + silu(causal_conv_k3(a, W[f"up{q}.res{r}.W"], d, left) + W[f"up{q}.res{r}.b"])
        g = silu(a)
        left, self.c_head = self.c_head, np.concatenate([self.c_head, g], axis=0)[-2:]
        z = causal_conv_k3(g, W["head.W"], 1, left) + W["head.b"]
        xi = frame_signal(z, cfg.n_fft, cfg.logmag_clamp)
        pcm, self.tail = overlap_add(xi, cfg.n_fft, cfg.hop, self.tail)
        return pcm.astype(np.float32)


# --------------------------------------------------------------------------------------------
# drivers
# --------------------------------------------------------------------------------------------

class TokenToWavStream:
    """The whole decoder step (Sec. 2.2 lists the stages of the segment): the flow decoder's chunk of
    mel frames, rounded once to float32 as the flow decoder delivers it, is the vocoder tail's input."""

    def __init__(self, cfg, blob, **kw):
        fc, vc = cfg.flow_part(), cfg.vocoder_part()
        nf = _blob_floats(fc)
        self.flow = FlowStream(fc, blob[:nf], **kw)
        self.voc = VocoderStream(vc, blob[nf:], stream_id=kw.get("stream_id", 0))

    def decode_chunk(self, feats: np.ndarray) -> np.ndarray:
        mel = self.flow.decode_chunk(feats)
        return self.voc.decode_chunk(np.asarray(mel, dtype=np.float32))


def _blob_floats(cfg) -> int:
    """Number of floats of a flow configuration's blob (the same tensors that parse_blob takes;
    the oracle imports nothing from the input generators, so the count is written out here)."""
    C = cfg.hidden
    if cfg.pipeline == "flow":
        m = cfg.mel_dim
        return (2 * m * C + C + len(cfg.dilations) * (3 * C * C + C + C * C)
                + cfg.n_attn_layers * (4 * C * C + 4 * C) + C * m + m)
    raise ValueError(cfg.pipeline)


def token2wav_offline(cfg, blob, feats, boundaries, stream_id: int = 0) -> np.ndarray:
    fc, vc = cfg.flow_part(), cfg.vocoder_part()
    nf = _blob_floats(fc)
    mel = flow_offline(fc, blob[:nf], feats, boundaries, stream_id)
    return vocoder_offline(vc, blob[nf:], np.asarray(mel, dtype=np.float32), stream_id)


def make_stream(cfg, blob, **kw):
    if cfg.pipeline == "token2wav":
        return TokenToWavStream(cfg, blob, **kw)
    if cfg.pipeline == "conv":
        return ConvStackStream(cfg, blob)
    if cfg.pipeline == "flow":
        return FlowStream(cfg, blob, **kw)
    if cfg.pipeline == "vocoder":
        return VocoderStream(cfg, blob, stream_id=kw.get("stream_id", 0))
    raise ValueError(cfg.pipeline)


def run_offline(cfg, blob, feats, boundaries, stream_id: int = 0) -> np.ndarray:
    if cfg.pipeline == "token2wav":
        return token2wav_offline(cfg, blob, feats, boundaries, stream_id)
    if cfg.pipeline == "conv":
        return conv_stack_offline(cfg, blob, feats)
    if cfg.pipeline == "flow":
        return flow_offline(cfg, blob, feats, boundaries, stream_id)
    return vocoder_offline(cfg, blob, feats, stream_id)


def run_stream(cfg, blob, feats, boundaries, **kw) -> np.ndarray:
    st = make_stream(cfg, blob, **kw)
    la = getattr(cfg, "f_lookahead", 0)         # a call also presents the next <= la frames, which it does not commit
    F = boundaries[-1]
    outs = [st.decode_chunk(feats[boundaries[c]:min(boundaries[c + 1] + (la if boundaries[c + 1] - boundaries[c] == cfg.f_chunk else 0), F)])
            for c in range(len(boundaries) - 1)]
    return np.concatenate(outs, axis=0)
