"""GPU parity of the whole decoder step (flow decoder feeding the vocoder tail inside one
dc_decode_chunk, the mel frames staying on the device), through the C ABI.

The vocoder tail is a strongly expanding map (exp of the log-magnitude channels): in the oracle
itself, mel frames that differ by 4e-3 of their RMS give PCM that differs by about 3e-2.  The
parity of the chain is therefore stated stage by stage, on the data each stage really sees:
  * the flow stage's mel frames against the oracle's flow decoder        (bf16 bar, 2e-2),
  * the PCM against the ORACLE's vocoder tail applied to the GPU's mel   (fp32 bar, 1e-4),
and the distance of the PCM to the oracle's end-to-end chain is bounded by E2E_BOUND, the tightest
round value that held on every case measured (2.7e-2 at full size, 2.9e-2, 3.4e-2 and 4.2e-2 on the
tiny cases) with the flow stage keeping every declared bf16 rounding (the composite builds its flow
decoder with the rounded RMS norm; with the folded norm the same cases gave 3.2e-2 to 4.6e-2).
The 2e-2 bar of the bf16 pipelines is NOT met end to end: the flow stage sits 4e-3 from the oracle
- fp32 accumulation against the oracle's float64 flips individual bf16 roundings - and the tail
multiplies that by 6 to 7."""
import numpy as np
import pytest
import torch

import dc_workloads as wl
from oracle import dc_oracle as orc

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2
TOL_F32 = 1e-4
E2E_BOUND = 5e-2
RAGGED = [0, 3, 13, 14, 24, 31, 41, 51, 52, 62, 72, 80]


@pytest.fixture(scope="module")
def dc():
    import paper_2609_35115_b200 as dc
    dc.load_library()
    return dc


def _gu():
    from tests import gpu_util
    return gpu_util


def _stagewise(dc, cfg, boundaries=None, e2e_bound=E2E_BOUND):
    gu = _gu()
    w = wl.make_workload(cfg, boundaries=[boundaries] if boundaries else None)
    s = w.streams[0]
    fc, vc = cfg.flow_part(), cfg.vocoder_part()
    nf = wl.blob_size(fc)
    # the chain through the library
    m = dc.Model(cfg, w.weights)
    pcm = gu.run_gpu_stream(m, s.feats, s.boundaries)
    if cfg.noise_seed or cfg.excitation_std > 0:       # a model's second stream draws another random sequence:
        m.destroy()                                    # the rerun is the first stream of a fresh model
        m = dc.Model(cfg, w.weights)
    pcm2 = gu.run_gpu_stream(m, s.feats, s.boundaries)
    m.destroy()
    assert np.array_equal(pcm, pcm2), "reruns differ"
    assert pcm.shape == (s.boundaries[-1] * cfg.out_per_frame,) and np.isfinite(pcm).all()
    # the flow stage alone, same weights: its output is what the chain hands to the vocoder tail
    mf = dc.Model(fc, w.weights[:nf], options=dc.OPT_ROUNDED_NORM)     # as the composite builds it
    mel = gu.run_gpu_stream(mf, s.feats, s.boundaries)
    mf.destroy()
    ref_mel = orc.run_stream(fc, w.weights[:nf], s.feats, s.boundaries)
    e_mel = gu.rel_err(mel, ref_mel)
    assert e_mel <= TOL_BF16, f"flow stage: {e_mel}"
    # vocoder tail of the oracle on the GPU's mel frames
    ref_pcm_stage = orc.run_stream(vc, w.weights[nf:], mel, s.boundaries)
    e_voc = gu.rel_err(pcm, ref_pcm_stage)
    assert e_voc <= TOL_F32, f"vocoder stage: {e_voc}"
    # end to end against the oracle's chain (see the module docstring)
    ref = orc.run_stream(cfg, w.weights, s.feats, s.boundaries)
    e_all = gu.rel_err(pcm, ref)
    print(f"{cfg.name}: flow stage {e_mel:.2e}, vocoder stage {e_voc:.2e}, end to end {e_all:.2e}")
    assert e_all <= e2e_bound
    return e_mel, e_voc, e_all


def test_tiny_chain_ragged(dc):
    _stagewise(dc, wl.tiny_token2wav(n_chunks=len(RAGGED) - 1), boundaries=RAGGED)


def test_token2wav_full_size(dc):
    """cfg3's flow decoder + cfg4's vocoder tail, 6 chunks of 50 frames (24,000 samples each)."""
    _stagewise(dc, wl.token2wav(n_chunks=6))


def test_chain_equals_the_two_models_by_hand(dc):
    """The composite is exactly the two pipelines chained on the device."""
    gu = _gu()
    cfg = wl.tiny_token2wav(n_chunks=5)
    w = wl.make_workload(cfg)
    s = w.streams[0]
    nf = wl.blob_size(cfg.flow_part())
    m = dc.Model(cfg, w.weights)
    pcm = gu.run_gpu_stream(m, s.feats, s.boundaries)
    m.destroy()
    mf, mv = dc.Model(cfg.flow_part(), w.weights[:nf], options=dc.OPT_ROUNDED_NORM), dc.Model(cfg.vocoder_part(), w.weights[nf:])
    sf, sv = mf.open_stream(), mv.open_stream()
    x = torch.from_numpy(s.feats).cuda()
    outs = []
    for c in range(len(s.boundaries) - 1):
        mel = sf.decode_chunk(x[s.boundaries[c]:s.boundaries[c + 1]].contiguous())
        outs.append(sv.decode_chunk(mel.contiguous()).clone())
    torch.cuda.synchronize()
    by_hand = torch.cat(outs).cpu().numpy()
    sf.close(); sv.close(); mf.destroy(); mv.destroy()
    assert np.array_equal(pcm, by_hand)


@pytest.mark.parametrize("n_streams", [3, 11])
def test_batched_chain_equals_single_stream(dc, n_streams):
    """The batch call runs the streams' vocoder tails side by side on CUDA streams of the model (8 at most:
    with 11 streams some side streams carry two tails); every stream's bytes are those of its own calls."""
    cfg = wl.tiny_token2wav(n_chunks=4, n_streams=n_streams)
    w = wl.make_workload(cfg)
    gu = _gu()
    m = dc.Model(cfg, w.weights, max_batch=n_streams)
    single = [gu.run_gpu_stream(m, s.feats, s.boundaries) for s in w.streams]
    streams = [m.open_stream() for _ in w.streams]
    feats = [torch.from_numpy(s.feats).cuda() for s in w.streams]
    outs = [torch.zeros(s.boundaries[-1] * cfg.out_per_frame, device="cuda") for s in w.streams]
    n_rounds = max(len(s.boundaries) - 1 for s in w.streams)
    for r in range(n_rounds):
        idx = [i for i, s in enumerate(w.streams) if r < len(s.boundaries) - 1]
        fs = [feats[i][w.streams[i].boundaries[r]:w.streams[i].boundaries[r + 1]].contiguous() for i in idx]
        os_ = [outs[i][w.streams[i].boundaries[r] * cfg.out_per_frame:w.streams[i].boundaries[r + 1] * cfg.out_per_frame] for i in idx]
        dc.decode_batch(m, [streams[i] for i in idx], fs, os_)
    torch.cuda.synchronize()
    assert m.counters()[4] == 0
    for st in streams:
        st.close()
    m.destroy()
    for i in range(len(w.streams)):
        assert np.array_equal(outs[i].cpu().numpy(), single[i]), f"stream {i}"


def test_chain_reset_and_carry_addresses(dc):
    gu = _gu()
    cfg = wl.tiny_token2wav(n_chunks=4)
    w = wl.make_workload(cfg)
    s = w.streams[0]
    m = dc.Model(cfg, w.weights)
    st = m.open_stream()
    before = st.carry_info()
    a = gu.run_gpu_stream(m, s.feats, s.boundaries, stream=st)
    assert st.carry_info() == before and len(before) > 4     # flow carries + vocoder rings, never moved
    st.reset()
    b = gu.run_gpu_stream(m, s.feats, s.boundaries, stream=st)
    st.close()
    m.destroy()
    assert np.array_equal(a, b)


def test_chain_with_device_randomness_in_both_stages(dc):
    """The whole decoder step drawing its own randomness: the flow decoder's Euler noise and the vocoder's
    excitation, both Philox streams keyed by the session and its clocks; stage-wise parity as above."""
    _stagewise(dc, wl.tiny_token2wav(n_chunks=len(RAGGED) - 1, noise_seed=41, excitation_std=0.2, excitation_seed=43), boundaries=RAGGED)


@pytest.mark.parametrize("make", [lambda: wl.tiny_token2wav(n_chunks=4, n_streams=3), lambda: wl.tiny_vocoder(n_chunks=4, n_streams=3)])
@pytest.mark.parametrize("pinned", [True, False])
def test_host_buffer_batch_call_serves_the_fp32_and_composite_pipelines(dc, make, pinned):
    """dc_decode_batch_host for the pipelines that stage through the model's bounce buffers: same bytes as the
    device-pointer batch call, with page-locked and with pageable caller buffers."""
    cfg = make()
    w = wl.make_workload(cfg)
    S = cfg.n_streams
    m = dc.Model(cfg, w.weights, max_batch=S)
    opf = cfg.out_per_frame

    def run(host):
        streams = [m.open_stream() for _ in range(S)]
        outs = []
        for r in range(cfg.n_chunks):
            lo, hi = w.streams[0].boundaries[r], w.streams[0].boundaries[r + 1]
            if host:
                fin = [torch.from_numpy(np.ascontiguousarray(s.feats[lo:hi])) for s in w.streams]
                fout = [torch.zeros((hi - lo) * opf) for _ in range(S)]
                if pinned:
                    fin, fout = [t.pin_memory() for t in fin], [t.pin_memory() for t in fout]
                dc.decode_batch_host(m, streams, fin, fout)
                outs.append(np.stack([t.numpy().copy() for t in fout]))
            else:
                fin = [torch.from_numpy(np.ascontiguousarray(s.feats[lo:hi])).cuda() for s in w.streams]
                fout = [torch.zeros((hi - lo) * opf, device="cuda") for _ in range(S)]
                dc.decode_batch(m, streams, fin, fout)
                torch.cuda.synchronize()
                outs.append(np.stack([t.cpu().numpy() for t in fout]))
        for st in streams:
            st.close()
        return np.concatenate(outs, axis=1)

    a, b = run(False), run(True)
    assert m.counters()[4] == 0
    m.destroy()
    assert np.isfinite(a).all() and np.array_equal(a, b)
