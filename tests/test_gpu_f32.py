"""GPU parity of the fp32 pipelines (tiny causal conv stream, vocoder tail) against the oracle,
through the C ABI.  Tolerance: max |err| / RMS(ref) <= 1e-4."""
import hashlib

import numpy as np
import pytest
import torch

import dc_workloads as wl
from oracle import dc_oracle as orc

pytestmark = pytest.mark.gpu

TOL_F32 = 1e-4


@pytest.fixture(scope="module")
def dc():
    import paper_2609_35115_b200 as dc
    dc.load_library()
    return dc


def _util():
    from tests import gpu_util
    return gpu_util


def test_cfg1_streamed_matches_offline_oracle(dc):
    gu = _util()
    w = wl.make_workload(wl.CONFIGS["cfg1"])
    s = w.streams[0]
    ref = orc.run_offline(w.cfg, w.weights, s.feats, s.boundaries)
    m = dc.Model(w.cfg, w.weights)
    got = gu.run_gpu_stream(m, s.feats, s.boundaries)
    assert got.shape == ref.shape
    assert gu.rel_err(got, ref) <= TOL_F32
    # ragged partition incl. chunks shorter than the conv left context
    ragged = [0, 1, 2, 5, 21, 22, 38, 39, 55, 71, 87, 103, 119, 128]
    got2 = gu.run_gpu_stream(m, s.feats, ragged)
    assert gu.rel_err(got2, ref) <= TOL_F32
    # bitwise reproducible run to run
    got3 = gu.run_gpu_stream(m, s.feats, s.boundaries)
    assert hashlib.sha256(got.tobytes()).hexdigest() == hashlib.sha256(got3.tobytes()).hexdigest()
    m.destroy()


def test_conv_stack_nonzero_bias_large_dilation(dc):
    gu = _util()
    cfg = wl.CONFIGS["cfg1"].replace(name="conv_b", hidden=72, dilations=(1, 3, 9), f_chunk=40, n_chunks=6,
                                     seed=21, bias_std=0.3)
    bnd = [0, 40, 41, 60, 100, 117, 157]
    w = wl.make_workload(cfg, boundaries=[bnd])
    s = w.streams[0]
    ref = orc.run_offline(cfg, w.weights, s.feats, bnd)
    m = dc.Model(cfg, w.weights)
    assert gu.rel_err(gu.run_gpu_stream(m, s.feats, bnd), ref) <= TOL_F32
    m.destroy()


def test_tiny_vocoder_ragged_chunks(dc):
    gu = _util()
    cfg = wl.tiny_vocoder()
    bnd = [0, 1, 2, 7, 8, 13, 18, 20]
    w = wl.make_workload(cfg, boundaries=[bnd])
    s = w.streams[0]
    ref = orc.vocoder_offline(cfg, w.weights, s.feats)
    m = dc.Model(cfg, w.weights)
    got = gu.run_gpu_stream(m, s.feats, bnd)
    assert got.shape == ref.shape
    assert gu.rel_err(got, ref) <= TOL_F32
    m.destroy()


def test_cfg4_vocoder_tail_full(dc):
    gu = _util()
    cfg = wl.CONFIGS["cfg4"]
    w = wl.make_workload(cfg)
    s = w.streams[0]
    ref = orc.run_stream(cfg, w.weights, s.feats, s.boundaries)
    m = dc.Model(cfg, w.weights)
    got = gu.run_gpu_stream(m, s.feats, s.boundaries)
    assert got.shape == (cfg.n_chunks * 24000,)
    assert gu.rel_err(got, ref) <= TOL_F32
    # per chunk, too
    for c in (0, 1, 57, 199):
        assert gu.rel_err(got[c * 24000:(c + 1) * 24000], ref[c * 24000:(c + 1) * 24000]) <= TOL_F32
    got2 = gu.run_gpu_stream(m, s.feats, s.boundaries)
    assert np.array_equal(got, got2)
    m.destroy()


def test_vocoder_reset_and_pointer_constancy(dc):
    gu = _util()
    cfg = wl.tiny_vocoder()
    w = wl.make_workload(cfg)
    s = w.streams[0]
    m = dc.Model(cfg, w.weights)
    st = m.open_stream()
    before = st.carry_info()
    a = gu.run_gpu_stream(m, s.feats, s.boundaries, stream=st)
    assert st.carry_info() == before           # carries never move while the stream lives
    st.reset()
    assert st.carry_info() == before           # ... nor at a turn boundary
    b = gu.run_gpu_stream(m, s.feats, s.boundaries, stream=st)
    assert np.array_equal(a, b)                # reset writes the base state in place
    st.close()
    m.destroy()


def test_admission_and_error_paths(dc):
    cfg = wl.CONFIGS["cfg1"]
    w = wl.make_workload(cfg)
    m = dc.Model(cfg, w.weights)
    st = m.open_stream()
    x = torch.zeros(17, 64, device="cuda")
    y = torch.zeros(17, 64, device="cuda")
    good = torch.from_numpy(w.streams[0].feats[:16]).cuda()
    ref1 = st.decode_chunk(good).clone()
    # admission predicate: 1 <= n_frames <= f_chunk; a refused call must not touch the stream
    assert st.decode_raw(x.data_ptr(), 17, y.data_ptr()) == 3
    assert st.decode_raw(x.data_ptr(), 0, y.data_ptr()) == 3
    assert st.decode_raw(0, 4, y.data_ptr()) == 1
    assert st.decode_raw(x.data_ptr(), 4, 0) == 1
    nxt = torch.from_numpy(w.streams[0].feats[16:32]).cuda()
    got2 = st.decode_chunk(nxt).clone()
    ref = orc.run_offline(cfg, w.weights, w.streams[0].feats[:32], [0, 32])
    torch.cuda.synchronize()
    from tests import gpu_util as gu
    assert gu.rel_err(torch.cat([ref1, got2]).cpu().numpy(), ref) <= TOL_F32
    c = m.counters()
    assert c[0] == 2 and c[1] == 32 and c[2] == 2 and c[3] == 2 and c[5] == 6   # per chunk: call record + 2 conv blocks
    # a model with open streams cannot be destroyed; a closed stream refuses work
    with pytest.raises(dc.DCError):
        m.destroy()
    h = st.handle
    st.close()
    st.handle = h
    assert st.decode_raw(x.data_ptr(), 4, y.data_ptr()) == 7
    st.handle = None
    # bad configuration / blob size fail closed
    with pytest.raises(dc.DCError):
        dc.Model(cfg, w.weights[:-1])
    with pytest.raises(dc.DCError):
        dc.Model(cfg.replace(hidden=63), w.weights)
    m.destroy()


def test_host_buffer_entry_point(dc):
    gu = _util()
    cfg = wl.CONFIGS["cfg1"]
    w = wl.make_workload(cfg)
    s = w.streams[0]
    m = dc.Model(cfg, w.weights)
    st = m.open_stream()
    fin = torch.from_numpy(s.feats).pin_memory()
    fout = torch.empty(s.feats.shape[0], 64).pin_memory()
    for c in range(len(s.boundaries) - 1):
        lo, hi = s.boundaries[c], s.boundaries[c + 1]
        n = st.decode_chunk_host(fin[lo:hi], fout[lo:hi])
        assert n == (hi - lo) * 64
    ref = orc.run_offline(cfg, w.weights, s.feats, s.boundaries)
    assert gu.rel_err(fout.numpy(), ref) <= TOL_F32
    st.close()
    m.destroy()


def test_bounded_device_wait_gives_up_and_reports(dc):
    """A wait on a barrier that nothing completes runs out after its poll limit and the host reads
    DC_ERR_TIMEOUT; the context stays usable (a decode call works right after)."""
    assert dc.selftest_bounded_wait(1000) == 6           # DC_ERR_TIMEOUT: the wait gave up, as it must
    assert dc.selftest_bounded_wait(0) == 1              # argument check
    cfg = wl.CONFIGS["cfg1"]
    w = wl.make_workload(cfg)
    m = dc.Model(cfg, w.weights)
    st = m.open_stream()
    y = st.decode_chunk(torch.from_numpy(w.streams[0].feats[:16]).cuda())
    torch.cuda.synchronize()
    assert torch.isfinite(y).all()
    st.close()
    m.destroy()


def test_streams_of_one_model_on_different_cuda_streams(dc):
    """Each stream's captured chunk step reads a call record of its own, so two streams of one model may
    decode at the same time on different CUDA streams."""
    import torch
    from tests import gpu_util as gu
    cfg = wl.tiny_vocoder(n_chunks=6, n_streams=2)
    w = wl.make_workload(cfg)
    m = dc.Model(cfg, w.weights)
    ref = [gu.run_gpu_stream(m, s.feats, s.boundaries) for s in w.streams]
    sts = [m.open_stream() for _ in w.streams]
    cs = [torch.cuda.Stream() for _ in w.streams]
    xs = [torch.from_numpy(s.feats).cuda() for s in w.streams]
    outs = [[], []]
    torch.cuda.synchronize()
    n_rounds = max(len(s.boundaries) - 1 for s in w.streams)
    for r in range(n_rounds):
        for i, s in enumerate(w.streams):
            if r < len(s.boundaries) - 1:
                outs[i].append(sts[i].decode_chunk(xs[i][s.boundaries[r]:s.boundaries[r + 1]].contiguous(), stream=cs[i]))
    torch.cuda.synchronize()
    for i in range(2):
        got = torch.cat(outs[i]).cpu().numpy()
        assert np.array_equal(got, ref[i]), f"stream {i}"
        sts[i].close()
    m.destroy()


# ---- the vocoder's random excitation: drawn on the device, keyed by the stream and its output-frame clock ----

EXC = dict(excitation_std=0.25, excitation_seed=0xABCDEF0123)


def test_vocoder_excitation_matches_oracle_for_any_chunking_and_stream(dc):
    gu = _util()
    cfg = wl.tiny_vocoder(bias_std=0.3, **EXC)
    bnd = [0, 1, 2, 7, 8, 13, 18, 20]
    w = wl.make_workload(cfg, boundaries=[bnd])
    s = w.streams[0]
    m = dc.Model(cfg, w.weights)
    quiet = orc.vocoder_offline(cfg.replace(excitation_std=0.0), w.weights, s.feats)
    outs = []
    for sid, b in enumerate((bnd, [0, 5, 10, 15, 20], bnd)):       # the model's streams 0, 1, 2 draw different sequences
        ref = orc.vocoder_offline(cfg, w.weights, s.feats, stream_id=sid)
        st = m.open_stream()
        got = gu.run_gpu_stream(m, s.feats, b, stream=st)
        assert gu.rel_err(got, ref) <= TOL_F32, f"stream {sid}"
        assert gu.rel_err(got, quiet) > 1e-2                        # the source is really there
        outs.append(got)
        if sid == 2:                                                # a reset restarts the stream's clock: same draw again
            st.reset()
            assert np.array_equal(gu.run_gpu_stream(m, s.feats, b, stream=st), got)
        st.close()
    assert not np.array_equal(outs[0], outs[2])
    m.destroy()
    # direct launches draw what the captured chunk step draws
    m2 = dc.Model(cfg, w.weights, options=dc.OPT_NO_GRAPH)
    assert np.array_equal(gu.run_gpu_stream(m2, s.feats, bnd), outs[0])
    m2.destroy()


def test_vocoder_excitation_cfg4_geometry(dc):
    """cfg4's network with the excitation on: 6 chunks of 50 frames (6,000 excitation frames of 64 channels each)."""
    gu = _util()
    cfg = wl.CONFIGS["cfg4"].replace(name="cfg4_excited", n_chunks=6, **EXC)
    w = wl.make_workload(cfg)
    s = w.streams[0]
    ref = orc.run_stream(cfg, w.weights, s.feats, s.boundaries)
    m = dc.Model(cfg, w.weights)
    got = gu.run_gpu_stream(m, s.feats, s.boundaries)
    m.destroy()
    assert gu.rel_err(got, ref) <= TOL_F32


def test_excitation_needs_a_seed_and_a_vocoder(dc):
    cfg = wl.tiny_vocoder(excitation_std=0.2)                       # no seed
    w = wl.make_workload(cfg)
    with pytest.raises(dc.DCError):
        dc.Model(cfg, w.weights)
    c1 = wl.CONFIGS["cfg1"].replace(excitation_std=0.2, excitation_seed=3)
    with pytest.raises(dc.DCError):
        dc.Model(c1, wl.make_workload(c1).weights)


# ---- multi-stream batching of the fp32 pipelines: every layer one launch for all the streams of the batch ----

@pytest.mark.parametrize("make", [lambda: wl.tiny_vocoder(n_streams=5, n_chunks=6, bias_std=0.2, **EXC),
                                  lambda: wl.CONFIGS["cfg1"].replace(name="cfg1_batch", n_streams=3, bias_std=0.2),
                                  lambda: wl.CONFIGS["cfg4"].replace(name="cfg4_batch", n_streams=4, n_chunks=3)])
def test_f32_batched_streams_equal_single_stream_bytes_and_oracle(dc, make):
    gu = _util()
    cfg = make()
    S = cfg.n_streams
    bounds = None
    if cfg.f_chunk <= 16:      # ragged and different per stream (a stream that has run out of chunks sits a round out)
        F = cfg.f_chunk * cfg.n_chunks
        rng = np.random.default_rng(3)
        bounds = []
        for _ in range(S):
            b = [0]
            while b[-1] < F:
                b.append(min(F, b[-1] + int(rng.integers(1, cfg.f_chunk + 1))))
            bounds.append(b)
    w = wl.make_workload(cfg, boundaries=bounds)
    # single-stream runs on a model of their own, so that stream i is that model's i-th stream here too
    m1 = dc.Model(cfg, w.weights)
    single = []
    for s in w.streams:
        st = m1.open_stream()
        single.append(gu.run_gpu_stream(m1, s.feats, s.boundaries, stream=st))
        st.close()
    m1.destroy()
    m = dc.Model(cfg, w.weights, max_batch=S)
    streams = [m.open_stream() for _ in range(S)]
    feats = [torch.from_numpy(s.feats).cuda() for s in w.streams]
    outs = [torch.zeros(s.boundaries[-1] * cfg.out_per_frame, device="cuda") for s in w.streams]
    opf = cfg.out_per_frame
    c0 = m.counters()
    rounds = max(len(s.boundaries) - 1 for s in w.streams)
    calls = 0
    for r in range(rounds):
        idx = [i for i, s in enumerate(w.streams) if r < len(s.boundaries) - 1]
        fs = [feats[i][w.streams[i].boundaries[r]:w.streams[i].boundaries[r + 1]] for i in idx]
        os_ = [outs[i][w.streams[i].boundaries[r] * opf:w.streams[i].boundaries[r + 1] * opf] for i in idx]
        dc.decode_batch(m, [streams[i] for i in idx], fs, os_)
        calls += 1
    torch.cuda.synchronize()
    c1 = m.counters()
    assert c1[7] - c0[7] == calls                         # one graph launch per round, whoever is present
    for st in streams:
        st.close()
    m.destroy()
    for i, s in enumerate(w.streams):
        got = outs[i].cpu().numpy().reshape(single[i].shape)
        assert np.array_equal(got, single[i]), f"{cfg.name}: stream {i} differs from its single-stream bytes"
        if i < 2:
            ref = orc.run_stream(cfg, w.weights, s.feats, s.boundaries, stream_id=i)
            assert gu.rel_err(got, ref) <= TOL_F32
