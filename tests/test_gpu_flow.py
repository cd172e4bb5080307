"""GPU parity of the bf16 flow decoder (conv blocks + chunk-causal attention + Euler steps)
against the bf16-mirrored oracle, through the C ABI.  Tolerance: max |err| / RMS(ref) <= 2e-2."""
import numpy as np
import pytest
import torch

import dc_workloads as wl
from oracle import dc_oracle as orc

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2
RAGGED = [0, 3, 13, 14, 24, 31, 41, 51, 52, 62, 72, 80]      # T in {1,3,7,8,10}; wraps the K/V ring


@pytest.fixture(scope="module")
def dc():
    import paper_2609_35115_b200 as dc
    dc.load_library()
    return dc


def _gu():
    from tests import gpu_util
    return gpu_util


def _parity(dc, cfg, boundaries=None, tol=TOL_BF16):
    gu = _gu()
    w = wl.make_workload(cfg, boundaries=[boundaries] if boundaries else None)
    s = w.streams[0]
    ref = orc.run_stream(cfg, w.weights, s.feats, s.boundaries)
    m = dc.Model(cfg, w.weights)
    got = gu.run_gpu_stream(m, s.feats, s.boundaries)
    err = gu.rel_err(got, ref)
    got2 = gu.run_gpu_stream(m, s.feats, s.boundaries)
    m.destroy()
    assert got.shape == ref.shape
    assert np.isfinite(got).all()
    assert err <= tol, f"{cfg.name}: max|err|/rms = {err}"
    assert np.array_equal(got, got2), "not bitwise reproducible run to run"
    return err


def test_flow_conv_only_gemm_path(dc):
    # no attention: input projection, conv blocks with carried left context, Euler epilogue
    _parity(dc, wl.tiny_flow(name="tiny_conv_only", n_attn_layers=0, n_heads=0, head_dim=0, kv_cap=0,
                             dilations=(1, 2, 4)), RAGGED)


def test_flow_tiny_with_attention_ragged(dc):
    _parity(dc, wl.tiny_flow(), RAGGED)


def test_flow_tiny_head_dim_64_full_chunks(dc):
    _parity(dc, wl.tiny_flow(name="tiny_h64", hidden=128, n_heads=2, head_dim=64, kv_cap=150, f_chunk=50,
                             n_chunks=6, dilations=(1, 2, 4, 1), n_steps=2))


def test_cfg2_small_flow_decoder(dc):
    _parity(dc, wl.CONFIGS["cfg2"])


def test_cfg3_token2wav_sized_flow_decoder(dc):
    # the whole configuration, 100 chunks: passes the K/V cap (512 frames after 11 chunks) and wraps the
    # 562-row ring several times; _parity also asserts that a second full run gives the same bytes
    assert wl.CONFIGS["cfg3"].n_chunks == 100
    _parity(dc, wl.CONFIGS["cfg3"])


def test_batched_streams_match_oracle_and_single_stream_bytes(dc):
    gu = _gu()
    cfg = wl.tiny_flow(name="tiny_batch", n_streams=5, n_chunks=5)
    w = wl.make_workload(cfg)
    m = dc.Model(cfg, w.weights, max_batch=5)
    single = [gu.run_gpu_stream(m, s.feats, s.boundaries) for s in w.streams]
    streams = [m.open_stream() for _ in w.streams]
    feats = [torch.from_numpy(s.feats).cuda() for s in w.streams]
    outs = [torch.empty(s.feats.shape[0], cfg.mel_dim, device="cuda") for s in w.streams]
    for r in range(cfg.n_chunks):
        fs, os_, ss = [], [], []
        for i, s in enumerate(w.streams):
            lo, hi = s.boundaries[r], s.boundaries[r + 1]
            fs.append(feats[i][lo:hi])
            os_.append(outs[i][lo:hi])
            ss.append(streams[i])
        dc.decode_batch(m, ss, fs, os_)
    torch.cuda.synchronize()
    for i, s in enumerate(w.streams):
        got = outs[i].cpu().numpy()
        ref = orc.run_stream(cfg, w.weights, s.feats, s.boundaries)
        assert gu.rel_err(got, ref) <= TOL_BF16
        assert np.array_equal(got, single[i]), "batched result differs from the single-stream bytes"
    for st in streams:
        st.close()
    m.destroy()


def test_flow_reset_and_pointer_constancy(dc):
    gu = _gu()
    cfg = wl.tiny_flow()
    w = wl.make_workload(cfg)
    s = w.streams[0]
    m = dc.Model(cfg, w.weights)
    st = m.open_stream()
    before = st.carry_info()
    assert len(before) == 2
    a = gu.run_gpu_stream(m, s.feats, s.boundaries, stream=st)
    assert st.carry_info() == before
    st.reset()
    b = gu.run_gpu_stream(m, s.feats, s.boundaries, stream=st)
    assert st.carry_info() == before and np.array_equal(a, b)
    st.close()
    m.destroy()


def test_cfg5_multi_stream_serving_full_size(dc):
    """32 staggered streams x 100 chunks through dc_decode_batch (the launch configuration the
    benchmark times).  Sampled streams are checked against the oracle; every stream is checked
    against the property that batching does not change the bytes (prefix of 12 chunks)."""
    gu = _gu()
    cfg = wl.CONFIGS["cfg5"]
    w = wl.make_workload(cfg)
    S = cfg.n_streams
    assert len({s.boundaries[1] for s in w.streams}) > 8          # offsets really are staggered
    m = dc.Model(cfg, w.weights, max_batch=S)
    feats = [torch.from_numpy(s.feats).cuda() for s in w.streams]

    def full_run():
        streams = [m.open_stream() for _ in range(S)]
        outs = [torch.empty(s.feats.shape[0], cfg.mel_dim, device="cuda") for s in w.streams]
        for r in range(cfg.n_chunks):
            fs = [feats[i][w.streams[i].boundaries[r]:w.streams[i].boundaries[r + 1]] for i in range(S)]
            os_ = [outs[i][w.streams[i].boundaries[r]:w.streams[i].boundaries[r + 1]] for i in range(S)]
            dc.decode_batch(m, streams, fs, os_)
        torch.cuda.synchronize()
        assert m.counters()[4] == 0, "a bounded device-side wait timed out"
        for st in streams:
            st.close()
        return [o.cpu().numpy() for o in outs]

    got = full_run()
    assert all(np.isfinite(g).all() for g in got)
    again = full_run()
    assert all(np.array_equal(a, b) for a, b in zip(got, again)), "not bitwise reproducible run to run"
    # (a) four streams against the oracle: two over all 100 chunks, two over their first 40
    for i, n_ch in ((7, cfg.n_chunks), (20, cfg.n_chunks), (0, 40), (31, 40)):
        si = w.streams[i]
        b = si.boundaries[:n_ch + 1]
        ref = orc.run_stream(cfg, w.weights, si.feats[:b[-1]], b)
        err = gu.rel_err(got[i][:b[-1]], ref)
        assert err <= TOL_BF16, f"stream {i}: {err}"
    # (b) batching never changes a stream's bytes
    for i in (0, 13, 31):
        si = w.streams[i]
        b = si.boundaries[:13]
        single = gu.run_gpu_stream(m, si.feats[:b[-1]], b)
        assert np.array_equal(single, got[i][:b[-1]])
    m.destroy()


# ---- classifier-free guidance: two passes per Euler step, (1 + w) v_cond - w v_uncond ------------------

def test_guided_tiny_ragged(dc):
    _parity(dc, wl.tiny_flow(cfg_scale=0.7, n_chunks=len(RAGGED) - 1), boundaries=RAGGED)


def test_guided_head_dim_64_and_large_weight(dc):
    _parity(dc, wl.tiny_flow(cfg_scale=2.0, hidden=128, n_heads=2, head_dim=64, n_chunks=5))


def test_guided_cfg3_geometry(dc):
    """cfg3's network with guidance: the two passes fill the 128-row tiles that a single stream half uses."""
    _parity(dc, wl.CONFIGS["cfg3"].replace(name="cfg3_guided", cfg_scale=0.7, n_chunks=14))


def test_guided_batched_equals_single_stream(dc):
    gu = _gu()
    cfg = wl.tiny_flow(cfg_scale=0.7, n_chunks=5, n_streams=3)
    w = wl.make_workload(cfg)
    m = dc.Model(cfg, w.weights, max_batch=3)
    single = [gu.run_gpu_stream(m, s.feats, s.boundaries) for s in w.streams]
    streams = [m.open_stream() for _ in w.streams]
    feats = [torch.from_numpy(s.feats).cuda() for s in w.streams]
    outs = [torch.zeros(s.boundaries[-1], cfg.mel_dim, device="cuda") for s in w.streams]
    n_rounds = max(len(s.boundaries) - 1 for s in w.streams)
    for r in range(n_rounds):
        idx = [i for i, s in enumerate(w.streams) if r < len(s.boundaries) - 1]
        fs = [feats[i][w.streams[i].boundaries[r]:w.streams[i].boundaries[r + 1]].contiguous() for i in idx]
        os_ = [outs[i][w.streams[i].boundaries[r]:w.streams[i].boundaries[r + 1]] for i in idx]
        dc.decode_batch(m, [streams[i] for i in idx], fs, os_)
    torch.cuda.synchronize()
    assert m.counters()[4] == 0
    for st in streams:
        st.close()
    m.destroy()
    for i in range(len(w.streams)):
        assert np.array_equal(outs[i].cpu().numpy(), single[i]), f"stream {i}"


# ---- prompt + retained carry: the first f_prompt frames are never evicted, behind them a window of kv_cap frames ----

def test_prompt_carry_tiny_ragged(dc):
    """A chunk straddles the end of the prompt (frames 14..23, f_prompt = 17); the ring wraps several times."""
    _parity(dc, wl.tiny_flow(f_prompt=17, n_chunks=len(RAGGED) - 1), boundaries=RAGGED)


def test_prompt_carry_with_guidance(dc):
    _parity(dc, wl.tiny_flow(f_prompt=9, cfg_scale=0.7, n_chunks=len(RAGGED) - 1), boundaries=RAGGED)


def test_paper_operating_point_carry(dc):
    """cfg3's network with the paper's clock quantities: f_prompt = 302, f_retained = 100, 50-frame chunks
    (attended extents 302 / 352 / 402 once the prompt is in)."""
    cfg = wl.EXTRA_CONFIGS["cfg3_paper_carry"].replace(n_chunks=13)
    bounds = [0, 50, 100, 150, 200, 250, 300, 302, 352, 402, 452, 502, 552, 602]
    _parity(dc, cfg, boundaries=bounds)


# ---- look-ahead frames: a full call presents f_chunk + f_lookahead frames and commits the first f_chunk ----

LA_BOUNDS = [0, 10, 20, 30, 33, 43, 53, 63, 73, 80]          # f_chunk = 10: full calls (with look-ahead) and partial ones


def test_lookahead_tiny(dc):
    _parity(dc, wl.tiny_flow(f_lookahead=3, n_chunks=len(LA_BOUNDS) - 1), boundaries=LA_BOUNDS)


def test_lookahead_with_prompt_and_guidance(dc):
    _parity(dc, wl.tiny_flow(f_lookahead=3, f_prompt=17, cfg_scale=0.7, n_chunks=len(LA_BOUNDS) - 1), boundaries=LA_BOUNDS)


def test_paper_operating_point_full(dc):
    """The paper's declaration for this decoder: f_prompt = 302, f_retained = 100, f_chunk = 50, f_call = 56
    (6 look-ahead frames), n_steps = 10 - on cfg3's network; envelope 402 + 56 = 458 attended frames."""
    cfg = wl.EXTRA_CONFIGS["cfg3_paper"].replace(n_chunks=13)
    bounds = [0, 50, 100, 150, 200, 250, 300, 302, 352, 402, 452, 502, 552, 602]
    _parity(dc, cfg, boundaries=bounds)


# ---- device-drawn Euler noise (Philox keyed by the stream's frame clock) ----

def _noise_run(dc, m, cfg, w, s, stream_id):
    gu = _gu()
    got = gu.run_gpu_stream(m, s.feats, s.boundaries)          # opens the model's next stream
    ref = orc.run_stream(cfg, w.weights, s.feats, s.boundaries, stream_id=stream_id)
    err = gu.rel_err(got, ref)
    assert err <= TOL_BF16, f"{cfg.name} stream {stream_id}: {err}"
    return got


def test_device_noise_per_stream_and_replay(dc):
    import os
    cfg = wl.tiny_flow(noise_seed=0x1234567890ABCDEF, n_chunks=len(RAGGED) - 1)
    w = wl.make_workload(cfg, boundaries=[RAGGED])
    s = w.streams[0]
    assert s.feats.shape[1] == cfg.mel_dim                      # the input is the conditioning alone
    m = dc.Model(cfg, w.weights)
    a = _noise_run(dc, m, cfg, w, s, 0)
    b = _noise_run(dc, m, cfg, w, s, 1)                         # the model's second stream draws another sequence
    assert not np.array_equal(a, b)
    m.destroy()
    # a model that launches its kernels directly (no captured graph) draws exactly the same
    m2 = dc.Model(cfg, w.weights, options=dc.OPT_NO_GRAPH)
    assert np.array_equal(_noise_run(dc, m2, cfg, w, s, 0), a)
    m2.destroy()


def test_device_noise_with_lookahead_prompt_and_guidance(dc):
    cfg = wl.tiny_flow(noise_seed=77, f_lookahead=3, f_prompt=17, cfg_scale=0.7, n_chunks=len(LA_BOUNDS) - 1)
    w = wl.make_workload(cfg, boundaries=[LA_BOUNDS])
    m = dc.Model(cfg, w.weights)
    _noise_run(dc, m, cfg, w, w.streams[0], 0)
    m.destroy()


# ---- host-buffer batch call: page-locked caller buffers are accessed by the kernels directly, pageable ones
# ---- go through the model's bounce buffers; the bytes are those of the device-buffer call either way ----

@pytest.mark.parametrize("pinned_in,pinned_out", [(True, True), (False, False), (True, False), (False, True)])
def test_batch_host_pinned_and_pageable(dc, pinned_in, pinned_out):
    cfg = wl.tiny_flow(n_streams=3, n_chunks=5)
    w = wl.make_workload(cfg)
    gu = _gu()
    m = dc.Model(cfg, w.weights, max_batch=3)
    single = [gu.run_gpu_stream(m, s.feats, s.boundaries) for s in w.streams]
    streams = [m.open_stream() for _ in w.streams]
    outs = [[] for _ in w.streams]
    n_rounds = max(len(s.boundaries) - 1 for s in w.streams)
    for r in range(n_rounds):
        idx = [i for i, s in enumerate(w.streams) if r < len(s.boundaries) - 1]
        fs, os_ = [], []
        for i in idx:
            b = w.streams[i].boundaries
            f = torch.from_numpy(np.ascontiguousarray(w.streams[i].feats[b[r]:b[r + 1]]))
            o = torch.full((b[r + 1] - b[r], cfg.mel_dim), float("nan"))
            fs.append(f.pin_memory() if pinned_in else f)
            os_.append(o.pin_memory() if pinned_out else o)
        dc.decode_batch_host(m, [streams[i] for i in idx], fs, os_)     # returns after the results are in place
        for i, o in zip(idx, os_):
            outs[i].append(o.clone())
    assert m.counters()[4] == 0
    for st in streams:
        st.close()
    m.destroy()
    for i in range(len(w.streams)):
        assert np.array_equal(torch.cat(outs[i]).numpy(), single[i]), f"stream {i}"


@pytest.mark.parametrize("pinned", [True, False])
def test_chunk_host_pinned_and_pageable(dc, pinned):
    cfg = wl.tiny_flow(n_chunks=5)
    w = wl.make_workload(cfg)
    s = w.streams[0]
    m = dc.Model(cfg, w.weights)
    ref = _gu().run_gpu_stream(m, s.feats, s.boundaries)
    st = m.open_stream()
    fin = torch.from_numpy(s.feats)
    fout = torch.full((s.feats.shape[0], cfg.mel_dim), float("nan"))
    if pinned:
        fin, fout = fin.pin_memory(), fout.pin_memory()
    for c in range(len(s.boundaries) - 1):
        lo, hi = s.boundaries[c], s.boundaries[c + 1]
        n = st.decode_chunk_host(fin[lo:hi], fout[lo:hi])
        assert n == (hi - lo) * cfg.mel_dim
    st.close()
    m.destroy()
    assert np.array_equal(fout.numpy(), ref)


def test_partial_batch_is_one_graph_launch(dc):
    """A serving round in which some streams have nothing to decode: every admitted call is still ONE graph
    launch (counters[7]) - the chunk step of a batch size met for the first time is captured at that call -
    and gives the bytes of single-stream decoding."""
    gu = _gu()
    cfg = wl.tiny_flow(name="tiny_partial", n_streams=5, n_chunks=4)
    w = wl.make_workload(cfg)
    m = dc.Model(cfg, w.weights, max_batch=5)
    single = [gu.run_gpu_stream(m, s.feats, s.boundaries) for s in w.streams]
    streams = [m.open_stream() for _ in w.streams]
    feats = [torch.from_numpy(s.feats).cuda() for s in w.streams]
    outs = [torch.zeros(s.feats.shape[0], cfg.mel_dim, device="cuda") for s in w.streams]
    done = [0] * 5
    # rounds with 5, 3, 4, 2, ... streams present: every stream still sees its chunks in order
    present = [[0, 1, 2, 3, 4], [0, 2, 4], [1, 3], [0, 1, 2, 3], [4, 1, 3, 0, 2], [2, 4], [0, 1, 3], [2, 4]]
    for idx in present:
        idx = [i for i in idx if done[i] < cfg.n_chunks]
        if not idx:
            continue
        c0 = m.counters()
        fs = [feats[i][w.streams[i].boundaries[done[i]]:w.streams[i].boundaries[done[i] + 1]] for i in idx]
        os_ = [outs[i][w.streams[i].boundaries[done[i]]:w.streams[i].boundaries[done[i] + 1]] for i in idx]
        dc.decode_batch(m, [streams[i] for i in idx], fs, os_)
        c1 = m.counters()
        assert c1[7] == c0[7] + 1, f"batch of {len(idx)}: not a single graph launch"
        assert c1[5] > c0[5]
        for i in idx:
            done[i] += 1
    torch.cuda.synchronize()
    assert done == [cfg.n_chunks] * 5 and m.counters()[4] == 0
    for st in streams:
        st.close()
    m.destroy()
    for i in range(5):
        assert np.array_equal(outs[i].cpu().numpy(), single[i]), f"stream {i}"


def test_rounded_norm_option_matches_oracle_and_batching(dc):
    """DC_OPT_ROUNDED_NORM: the normalised activations stored and rounded to bf16 by a kernel of their own (the
    storage-point reading taken literally) instead of a scale folded into the projection's accumulator."""
    gu = _gu()
    cfg = wl.tiny_flow(name="tiny_rounded", n_streams=3, n_chunks=5)
    w = wl.make_workload(cfg)
    m = dc.Model(cfg, w.weights, max_batch=3, options=dc.OPT_ROUNDED_NORM)
    single = [gu.run_gpu_stream(m, s.feats, s.boundaries) for s in w.streams]
    for s, got in zip(w.streams, single):
        assert gu.rel_err(got, orc.run_stream(cfg, w.weights, s.feats, s.boundaries)) <= TOL_BF16
    streams = [m.open_stream() for _ in w.streams]
    feats = [torch.from_numpy(s.feats).cuda() for s in w.streams]
    outs = [torch.zeros(s.feats.shape[0], cfg.mel_dim, device="cuda") for s in w.streams]
    for r in range(cfg.n_chunks):
        dc.decode_batch(m, streams, [feats[i][w.streams[i].boundaries[r]:w.streams[i].boundaries[r + 1]] for i in range(3)],
                        [outs[i][w.streams[i].boundaries[r]:w.streams[i].boundaries[r + 1]] for i in range(3)])
    torch.cuda.synchronize()
    assert m.counters()[4] == 0
    for st in streams:
        st.close()
    m.destroy()
    for i in range(3):
        assert np.array_equal(outs[i].cpu().numpy(), single[i])
    # the two forms of the norm are different roundings of the same network, not different networks
    m0 = dc.Model(cfg, w.weights)
    folded = gu.run_gpu_stream(m0, w.streams[0].feats, w.streams[0].boundaries)
    m0.destroy()
    assert not np.array_equal(folded, single[0]) and gu.rel_err(folded, single[0].astype(np.float64)) <= TOL_BF16


def test_cta_pairs_option_same_bytes_as_single_ctas(dc):
    """DC_OPT_CTA_PAIRS: the conv and QKV GEMMs of a full batch as 256-row products on pairs of SMs
    (tcgen05 cta_group::2, each CTA staging half of the weight tile).  Same accumulators, same summation
    order: the bytes must be those of the default single-CTA launches, ragged chunks and carried state
    included; the profile classes prove that the paired kernels are what ran."""
    import dataclasses
    cfg = dataclasses.replace(wl.CONFIGS["cfg5"], name="cfg5_pairs", n_streams=24, n_chunks=6)
    w = wl.make_workload(cfg)
    S = cfg.n_streams
    feats = [torch.from_numpy(s.feats).cuda() for s in w.streams]

    def run(options, profiled_round=None):
        m = dc.Model(cfg, w.weights, max_batch=S, options=options)
        streams = [m.open_stream() for _ in range(S)]
        outs = [torch.zeros(s.feats.shape[0], cfg.mel_dim, device="cuda") for s in w.streams]
        launches = None
        for r in range(cfg.n_chunks):
            fs = [feats[i][w.streams[i].boundaries[r]:w.streams[i].boundaries[r + 1]] for i in range(S)]
            os_ = [outs[i][w.streams[i].boundaries[r]:w.streams[i].boundaries[r + 1]] for i in range(S)]
            if r == profiled_round:
                m.profile_begin()
            dc.decode_batch(m, streams, fs, os_)
            if r == profiled_round:
                launches = m.profile_end()[1]
        torch.cuda.synchronize()
        assert m.counters()[4] == 0, "a bounded device-side wait timed out"
        for st in streams:
            st.close()
        m.destroy()
        return [o.cpu().numpy() for o in outs], launches

    base, n_base = run(0, profiled_round=2)
    pairs, n_pairs = run(dc.OPT_CTA_PAIRS, profiled_round=2)
    per_step = len(cfg.dilations) + cfg.n_attn_layers
    assert n_base["gemm_pair"] == 0 and n_pairs["gemm_pair"] == cfg.n_steps * per_step
    assert n_pairs["gemm_conv"] == 0
    assert all(np.isfinite(p).all() for p in pairs)
    for i in range(S):
        assert np.array_equal(base[i], pairs[i]), f"stream {i}"
    # ... and a batch with an odd number of row tiles falls back to single CTAs
    cfg_odd = dataclasses.replace(cfg, name="cfg5_pairs_odd", n_streams=22)
    m = dc.Model(cfg_odd, w.weights, max_batch=22, options=dc.OPT_CTA_PAIRS)
    streams = [m.open_stream() for _ in range(22)]
    outs = [torch.zeros(50, cfg.mel_dim, device="cuda") for _ in range(22)]
    m.profile_begin()
    dc.decode_batch(m, streams, [feats[i][:50] for i in range(22)], outs)
    n_odd = m.profile_end()[1]
    assert n_odd["gemm_pair"] == 0 and n_odd["gemm_conv"] == cfg.n_steps * len(cfg.dilations)
    for st in streams:
        st.close()
    m.destroy()
