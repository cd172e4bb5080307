"""Host-side fault injection and the guard zones around a stream's device buffers.

Nothing here faults, traps or hangs the GPU: an injected allocation failure never reaches the device, and the
guard zones are ordinary device memory of the library's own allocations that the test reads and (in one case)
overwrites with a plain cudaMemset."""
import numpy as np
import pytest
import torch

import dc_workloads as wl

pytestmark = pytest.mark.gpu

RAGGED = [0, 3, 13, 14, 24, 31, 41, 51, 52, 62, 72, 80]


@pytest.fixture(scope="module")
def dc():
    import paper_2609_35115_b200 as dc
    dc.load_library()
    return dc


def _run(m, s, bounds, st):
    from tests import gpu_util as gu
    return gu.run_gpu_stream(m, s.feats, bounds, stream=st)


@pytest.mark.parametrize("make,bounds", [
    (lambda: wl.tiny_flow(f_prompt=17, cfg_scale=0.7, n_chunks=len(RAGGED) - 1), RAGGED),      # K/V ring wraps several times
    (lambda: wl.tiny_flow(f_lookahead=3, n_chunks=6), [0, 10, 20, 30, 33, 43, 50]),             # look-ahead rows past the ring head
    (lambda: wl.tiny_vocoder(n_chunks=8, excitation_std=0.2, excitation_seed=5), None),
    (lambda: wl.CONFIGS["cfg1"], None),
    (lambda: wl.tiny_token2wav(n_chunks=len(RAGGED) - 1), RAGGED),
    (lambda: wl.CONFIGS["cfg3"].replace(n_chunks=14), None),                                      # past the K/V cap at full width
])
def test_no_kernel_writes_outside_a_stream_buffer(dc, make, bounds):
    cfg = make()
    w = wl.make_workload(cfg, boundaries=[bounds] if bounds else None)
    s = w.streams[0]
    plain = dc.Model(cfg, w.weights)
    ref = _run(plain, s, s.boundaries, None)
    plain.destroy()
    m = dc.Model(cfg, w.weights, options=dc.OPT_GUARD_ZONES)
    st = m.open_stream()
    got = _run(m, s, s.boundaries, st)
    assert st.check_guards() == 0, "a kernel wrote outside a carry / ring / staging buffer"
    assert np.array_equal(got, ref)                     # the guard zones change no byte of the result
    assert m.counters()[4] == 0
    st.close()
    m.destroy()


def test_guard_check_detects_an_overwritten_zone(dc):
    try:
        from cuda.bindings import runtime as cudart
    except ImportError:
        from cuda import cudart
    cfg = wl.tiny_vocoder()
    w = wl.make_workload(cfg)
    m = dc.Model(cfg, w.weights, options=dc.OPT_GUARD_ZONES)
    st = m.open_stream()
    assert st.check_guards() == 0
    addr, nbytes = st.carry_info()[1]
    # one byte just behind the second ring, then one just in front of it: both are inside the library's own allocation
    (err,) = cudart.cudaMemset(addr + nbytes + 3, 0, 1)
    assert int(err) == 0
    assert st.check_guards() == 1
    (err,) = cudart.cudaMemset(addr - 1, 0, 1)
    assert int(err) == 0
    assert st.check_guards() == 2
    st.close()
    m.destroy()
    # a model without guard zones has nothing to check
    m2 = dc.Model(cfg, w.weights)
    st2 = m2.open_stream()
    assert st2.check_guards() == 0
    st2.close()
    m2.destroy()


@pytest.mark.parametrize("make", [lambda: wl.tiny_flow(), lambda: wl.tiny_vocoder(), lambda: wl.tiny_token2wav(),
                                  lambda: wl.CONFIGS["cfg3"].replace(n_chunks=2)])
def test_injected_allocation_failures_unwind_cleanly(dc, make):
    """Every device allocation of dc_create and dc_stream_open is made to fail in turn: the call reports DC_ERR_OOM,
    releases what it had allocated, and the same call succeeds right afterwards."""
    cfg = make()
    w = wl.make_workload(cfg)
    s = w.streams[0]
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    failures = 0
    for nth in range(1, 200):
        dc.fail_allocation(nth)
        m = st = None
        try:
            m = dc.Model(cfg, w.weights, max_batch=2, max_wave_frames=20 if cfg.pipeline == "token2wav" else 0)
            st = m.open_stream()
        except dc.DCError as e:
            failures += 1
            assert e.status == 4, f"allocation {nth}: {e}"          # DC_ERR_OOM
        finally:
            dc.fail_allocation(0)
        if st is not None:
            st.close()
        if m is not None:
            m.destroy()
        if m is not None and st is not None:
            break                                                   # nth is beyond the number of allocations
    else:
        raise AssertionError("more than 200 allocations?")
    assert failures >= 3
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 >= free0 - (8 << 20), f"device memory leaked over {failures} failed attempts: {(free0 - free1) >> 20} MiB"
    # and the library works as before
    from tests import gpu_util as gu
    m = dc.Model(cfg, w.weights)
    a = gu.run_gpu_stream(m, s.feats, s.boundaries)
    m.destroy()
    assert np.isfinite(a).all()


@pytest.mark.parametrize("make", [lambda: wl.tiny_flow(n_streams=5, n_chunks=6, cfg_scale=0.7),
                                  lambda: wl.tiny_vocoder(n_streams=5, n_chunks=6, excitation_std=0.2, excitation_seed=5),
                                  lambda: wl.tiny_token2wav(n_streams=3, n_chunks=6)])
def test_no_batched_or_wavefront_kernel_writes_outside_a_stream_buffer(dc, make):
    """The multi-stream launches (slot tables, batched fp32 layers) and the wavefront passes under guard zones."""
    cfg = make()
    w = wl.make_workload(cfg)
    S = cfg.n_streams
    is_flow = cfg.pipeline in ("flow", "token2wav")
    F = w.streams[0].feats.shape[0]
    m = dc.Model(cfg, w.weights, max_batch=max(S, cfg.n_steps if is_flow else 1), max_wave_frames=F if cfg.pipeline == "token2wav" else 0,
                 options=dc.OPT_GUARD_ZONES)
    streams = [m.open_stream() for _ in range(S)]
    feats = [torch.from_numpy(s.feats).cuda() for s in w.streams]
    opf = cfg.out_per_frame
    outs = [torch.zeros(F * opf, device="cuda") for _ in range(S)]
    for r in range(cfg.n_chunks):
        idx = [i for i in range(S) if (i + r) % 4 != 3]            # a different subset of the streams every round
        # (streams that sit a round out fall behind; give every present stream ITS next chunk)
        fs, os_ = [], []
        for i in idx:
            k = getattr(streams[i], "_next", 0)
            lo, hi = w.streams[i].boundaries[k], w.streams[i].boundaries[k + 1]
            fs.append(feats[i][lo:hi])
            os_.append(outs[i][lo * opf:hi * opf])
            streams[i]._next = k + 1
        dc.decode_batch(m, [streams[i] for i in idx], fs, os_)
    torch.cuda.synchronize()
    assert all(st.check_guards() == 0 for st in streams)
    if is_flow:                                                     # ... and one wavefront call over a stream's remaining input
        st = streams[0]
        k = st._next
        lo = w.streams[0].boundaries[k]
        if lo < F:
            st.decode_wavefront(feats[0][lo:].contiguous())
            torch.cuda.synchronize()
            assert st.check_guards() == 0
    assert m.counters()[4] == 0
    for st in streams:
        st.close()
    m.destroy()
