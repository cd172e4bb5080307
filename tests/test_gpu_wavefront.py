"""Wavefront decoding (dc_decode_wavefront): all of a stream's input in one call, n_steps chunks in flight,
one per Euler step.  The bar is the strictest there is: the bytes of the same chunks decoded one by one
through dc_decode_chunk (which the other test files hold against the oracle), the stream's carries included -
checked by decoding on after the wavefront call.  One case also goes against the oracle directly."""
import numpy as np
import pytest
import torch

import dc_workloads as wl
from oracle import dc_oracle as orc

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2


@pytest.fixture(scope="module")
def dc():
    import paper_2609_35115_b200 as dc
    dc.load_library()
    return dc


def _gu():
    from tests import gpu_util
    return gpu_util


def _uniform(n_frames, f_chunk):
    return list(range(0, n_frames, f_chunk)) + [n_frames]


def _wave_vs_chunks(dc, cfg, n_frames, split=None, oracle=False):
    """Decodes frames [0, split) as a wavefront and the rest chunk by chunk (split = None: all as a wavefront,
    then one more wavefront call of what a second utterance would be), against chunk-by-chunk decoding."""
    gu = _gu()
    fc = cfg.f_chunk
    bounds = _uniform(n_frames, fc)
    w = wl.make_workload(cfg.replace(n_chunks=len(bounds) - 1), boundaries=[bounds])
    s = w.streams[0]
    m = dc.Model(cfg, w.weights, max_batch=cfg.n_steps)
    ref = gu.run_gpu_stream(m, s.feats, bounds)                      # stream 0 of the model, chunk by chunk
    st = m.open_stream()
    x = torch.from_numpy(np.ascontiguousarray(s.feats)).cuda()
    cut = n_frames if split is None else split
    assert cut % fc == 0 or cut == n_frames
    got = [st.decode_wavefront(x[:cut].contiguous()).clone()]
    if cut < n_frames:
        rest = [b for b in bounds if b >= cut]
        la = cfg.f_lookahead
        for c in range(len(rest) - 1):
            lo, hi = rest[c], rest[c + 1]
            if la and hi - lo == fc:
                hi = min(hi + la, n_frames)
            got.append(st.decode_chunk(x[lo:hi].contiguous()).clone())
    torch.cuda.synchronize()
    assert m.counters()[4] == 0, "a bounded device-side wait timed out"
    got = torch.cat([g.reshape(-1) if g.dim() == 1 else g for g in got], dim=0).cpu().numpy()
    st.close()
    m.destroy()
    assert got.shape == ref.shape and np.isfinite(got).all()
    assert np.array_equal(got, ref), f"{cfg.name}: wavefront differs from chunk-by-chunk decoding"
    if oracle:
        o = orc.run_stream(cfg, w.weights, s.feats, bounds)
        err = gu.rel_err(got, o)
        assert err <= TOL_BF16, f"{cfg.name}: {err}"
    return got


def test_tiny_wavefront_equals_chunks_and_oracle(dc):
    # 87 frames = 8 full chunks + 7: ramp-up, steady state, ramp-down, ragged tail; ring wraps (kv_cap 24)
    _wave_vs_chunks(dc, wl.tiny_flow(), 87, oracle=True)


def test_wavefront_shorter_than_the_pipeline(dc):
    # fewer chunks than Euler steps: the wavefront never fills
    _wave_vs_chunks(dc, wl.tiny_flow(), 14)
    _wave_vs_chunks(dc, wl.tiny_flow(), 5)


def test_wavefront_then_streaming_continues_from_its_carries(dc):
    _wave_vs_chunks(dc, wl.tiny_flow(), 87, split=50)


def test_wavefront_conv_only(dc):
    _wave_vs_chunks(dc, wl.tiny_flow(name="tiny_conv_only", n_attn_layers=0, n_heads=0, head_dim=0, kv_cap=0,
                                     dilations=(1, 2, 4)), 63)


def test_wavefront_guided_prompt_lookahead(dc):
    _wave_vs_chunks(dc, wl.tiny_flow(f_lookahead=3, f_prompt=17, cfg_scale=0.7), 87, oracle=True)
    # (a wavefront call sees no frames beyond its own, so its last chunk has no look-ahead: the split case
    # runs without look-ahead frames)
    _wave_vs_chunks(dc, wl.tiny_flow(f_prompt=17, cfg_scale=0.7), 87, split=40)


def test_wavefront_device_noise(dc):
    # a model's streams draw different sequences, so the chunk-by-chunk run and the wavefront run are each
    # the first stream of a model of their own
    gu = _gu()
    cfg = wl.tiny_flow(noise_seed=0xABCDEF0123, f_lookahead=3, n_chunks=9)
    bounds = _uniform(87, cfg.f_chunk)
    w = wl.make_workload(cfg, boundaries=[bounds])
    s = w.streams[0]
    m = dc.Model(cfg, w.weights, max_batch=cfg.n_steps)
    ref = gu.run_gpu_stream(m, s.feats, bounds)                      # stream 0
    m.destroy()
    m = dc.Model(cfg, w.weights, max_batch=cfg.n_steps)
    st = m.open_stream()                                             # stream 0 again
    got = st.decode_wavefront(torch.from_numpy(s.feats).cuda().contiguous()).cpu().numpy()
    assert m.counters()[4] == 0
    st.close()
    m.destroy()
    assert np.array_equal(got, ref)
    err = gu.rel_err(got, orc.run_stream(cfg, w.weights, s.feats, bounds, stream_id=0))
    assert err <= TOL_BF16, err


def test_wavefront_cfg3_size(dc):
    """cfg3's decoder (10 Euler steps, 50-frame chunks): 24 chunks + a 33-frame tail, 10 chunks in flight."""
    _wave_vs_chunks(dc, wl.CONFIGS["cfg3"], 24 * 50 + 33)


def test_wavefront_paper_operating_point(dc):
    """Prompt 302 + 100 retained + 6 look-ahead frames, 10 steps: wavefront over 16 chunks."""
    _wave_vs_chunks(dc, wl.EXTRA_CONFIGS["cfg3_paper"], 16 * 50)


def test_wavefront_token2wav(dc):
    gu = _gu()
    cfg = wl.tiny_token2wav()
    bounds = _uniform(87, cfg.f_chunk)
    w = wl.make_workload(cfg.replace(n_chunks=len(bounds) - 1), boundaries=[bounds])
    s = w.streams[0]
    m = dc.Model(cfg, w.weights, max_batch=cfg.n_steps, max_wave_frames=50)
    ref = gu.run_gpu_stream(m, s.feats, bounds)
    st = m.open_stream()
    x = torch.from_numpy(s.feats).cuda().contiguous()
    a = st.decode_wavefront(x[:50].contiguous()).clone()
    b = st.decode_wavefront(x[50:].contiguous()).clone()            # a second call: shorter, reuses the mel buffer
    torch.cuda.synchronize()
    assert m.counters()[4] == 0
    # the mel buffer of a wavefront call is sized at dc_stream_open: a longer call is refused, nothing touched
    before = m.counters()
    with pytest.raises(dc.DCError):
        st.decode_wavefront(x[:51].contiguous())
    after = m.counters()
    assert after[3] == before[3] + 1 and after[5] == before[5] and after[0] == before[0]
    st.close()
    m.destroy()
    assert np.array_equal(torch.cat([a, b]).cpu().numpy(), ref)


def test_wavefront_needs_room_for_n_steps_chunks(dc):
    cfg = wl.tiny_flow()
    w = wl.make_workload(cfg)
    s = w.streams[0]
    m = dc.Model(cfg, w.weights, max_batch=cfg.n_steps - 1)
    st = m.open_stream()
    x = torch.from_numpy(s.feats).cuda().contiguous()
    with pytest.raises(dc.DCError):
        st.decode_wavefront(x)
    # refused before anything ran: the stream still decodes, from its base state
    got = _gu().run_gpu_stream(m, s.feats, s.boundaries, stream=st)
    ref = _gu().run_gpu_stream(m, s.feats, s.boundaries)
    st.close()
    m.destroy()
    assert np.array_equal(got, ref)


def _batch_case(dc, cfg, lengths, tok2wav=False):
    """Several streams of different lengths decoded by one dc_decode_wavefront_batch call, each against its own
    chunk-by-chunk run."""
    gu = _gu()
    bounds = [_uniform(n, cfg.f_chunk) for n in lengths]
    cfgn = cfg.replace(n_streams=len(lengths), n_chunks=max(len(b) for b in bounds) - 1)
    w = wl.make_workload(cfgn, boundaries=bounds)
    m = dc.Model(cfgn, w.weights, max_batch=len(lengths) * cfg.n_steps, max_wave_frames=max(lengths) if tok2wav else 0)
    refs = [gu.run_gpu_stream(m, s.feats[:n], b) for s, n, b in zip(w.streams, lengths, bounds)]
    sts = [m.open_stream() for _ in lengths]
    xs = [torch.from_numpy(np.ascontiguousarray(s.feats[:n])).cuda() for s, n in zip(w.streams, lengths)]
    outs = dc.decode_wavefront_batch(m, sts, xs)
    torch.cuda.synchronize()
    assert m.counters()[4] == 0
    for i, (o, r) in enumerate(zip(outs, refs)):
        assert np.array_equal(o.cpu().numpy(), r), f"{cfg.name}: stream {i}"
    # one stream too many for the model's slots: refused, nothing touched
    if not tok2wav:
        extra = m.open_stream()
        with pytest.raises(dc.DCError):
            dc.decode_wavefront_batch(m, sts + [extra], xs + [xs[0]])
        extra.close()
    for st in sts:
        st.close()
    m.destroy()


def test_wavefront_batch_of_streams(dc):
    _batch_case(dc, wl.tiny_flow(), [87, 34, 120])


def test_wavefront_batch_guided_prompt_lookahead(dc):
    _batch_case(dc, wl.tiny_flow(f_lookahead=3, f_prompt=17, cfg_scale=0.7), [63, 87])


def test_wavefront_batch_token2wav(dc):
    _batch_case(dc, wl.tiny_token2wav(), [87, 34, 55], tok2wav=True)


def test_wavefront_batch_cfg3_size(dc):
    _batch_case(dc, wl.CONFIGS["cfg3"], [12 * 50, 9 * 50 + 20, 14 * 50 + 7])


def test_wavefront_direct_launches_equal_graph(dc):
    """The wavefront pass as direct launches (a model without graphs, and a profiled call) gives the bytes of
    the captured pass."""
    import os
    gu = _gu()
    cfg = wl.tiny_flow(f_prompt=17, cfg_scale=0.7)
    bounds = _uniform(87, cfg.f_chunk)
    w = wl.make_workload(cfg.replace(n_chunks=len(bounds) - 1), boundaries=[bounds])
    x = torch.from_numpy(w.streams[0].feats).cuda().contiguous()
    m = dc.Model(cfg, w.weights, max_batch=cfg.n_steps)
    st = m.open_stream()
    ref = st.decode_wavefront(x).cpu().numpy()
    st.reset()
    m.profile_begin(4096)
    got_prof = st.decode_wavefront(x).cpu().numpy()
    ms, nl = m.profile_end()
    assert sum(nl.values()) > 0
    st.close()
    m.destroy()
    m2 = dc.Model(cfg, w.weights, max_batch=cfg.n_steps, options=dc.OPT_NO_GRAPH)
    st2 = m2.open_stream()
    got_direct = st2.decode_wavefront(x).cpu().numpy()
    assert m2.counters()[4] == 0
    st2.close()
    m2.destroy()
    assert np.array_equal(got_prof, ref) and np.array_equal(got_direct, ref)


def test_wavefront_refusals_leave_the_streams_untouched(dc):
    """Argument errors of the wavefront calls are refused before anything runs."""
    gu = _gu()
    cfg = wl.tiny_flow()
    w = wl.make_workload(cfg)
    s = w.streams[0]
    m = dc.Model(cfg, w.weights, max_batch=2 * cfg.n_steps)
    other = dc.Model(cfg, w.weights, max_batch=cfg.n_steps)
    a, b, foreign = m.open_stream(), m.open_stream(), other.open_stream()
    x = torch.from_numpy(s.feats).cuda().contiguous()
    with pytest.raises(dc.DCError):                       # the same stream twice
        dc.decode_wavefront_batch(m, [a, a], [x, x])
    with pytest.raises(dc.DCError):                       # a stream of another model
        dc.decode_wavefront_batch(m, [a, foreign], [x, x])
    with pytest.raises(dc.DCError):                       # no frames
        dc.decode_wavefront_batch(m, [a], [x[:0].contiguous()])
    closed = m.open_stream()
    closed.close()
    with pytest.raises(dc.DCError):                       # a closed stream
        dc.decode_wavefront_batch(m, [closed], [x])
    # a vocoder model has no Euler loop to pipeline
    vcfg = wl.tiny_vocoder()
    vw = wl.make_workload(vcfg)
    vm = dc.Model(vcfg, vw.weights)
    vs = vm.open_stream()
    with pytest.raises(dc.DCError):
        vs.decode_wavefront(torch.from_numpy(vw.streams[0].feats).cuda().contiguous())
    vs.close()
    vm.destroy()
    # after all the refusals the two streams decode from their base state
    ref = gu.run_gpu_stream(m, s.feats, s.boundaries)
    got = dc.decode_wavefront_batch(m, [a, b], [x, x])
    torch.cuda.synchronize()
    assert m.counters()[4] == 0
    # (uniform chunks of the default workload: the wavefront cuts the same boundaries)
    assert s.boundaries == _uniform(s.boundaries[-1], cfg.f_chunk)
    for o in got:
        assert np.array_equal(o.cpu().numpy(), ref)
    for st in (a, b, foreign):
        st.close()
    m.destroy()
    other.destroy()
