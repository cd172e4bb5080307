"""dc_stream_snapshot / dc_stream_restore: a stream's carries and clocks, saved on the device and written
back in place - into the same stream (rewind) or into another stream of the same model (the session
moves).  After a restore the stream continues bit for bit as the original did."""
import numpy as np
import pytest
import torch

import dc_workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dc():
    import paper_2609_35115_b200 as dc
    dc.load_library()
    return dc


def _chunks(st, x, bounds, lo, hi):
    outs = [st.decode_chunk(x[bounds[c]:bounds[c + 1]].contiguous()).clone().reshape(-1) for c in range(lo, hi)]
    torch.cuda.synchronize()
    return torch.cat(outs).cpu().numpy()


@pytest.mark.parametrize("make", [lambda: wl.tiny_flow(n_chunks=8, f_prompt=9, cfg_scale=0.7),
                                  lambda: wl.tiny_flow(n_chunks=8, noise_seed=5),     # the session keeps its random stream

                                  lambda: wl.tiny_vocoder(n_chunks=8),
                                  lambda: wl.tiny_vocoder(n_chunks=8, excitation_std=0.3, excitation_seed=77),   # ... and its excitation clock
                                  lambda: wl.CONFIGS["cfg1"],
                                  lambda: wl.tiny_token2wav(n_chunks=8)])
def test_rewind_and_move(dc, make):
    cfg = make()
    w = wl.make_workload(cfg)
    s = w.streams[0]
    b = s.boundaries
    x = torch.from_numpy(s.feats).cuda()
    m = dc.Model(cfg, w.weights, max_batch=2)
    a = m.open_stream()
    addr = a.carry_info()
    _chunks(a, x, b, 0, 3)
    snap = a.snapshot()
    first = _chunks(a, x, b, 3, 6)
    a.restore(snap)                                   # rewind
    assert a.carry_info() == addr                     # in place
    again = _chunks(a, x, b, 3, 6)
    assert np.array_equal(first, again)
    other = m.open_stream()                           # move the session to another stream
    _chunks(other, x, b, 0, 2)                        # ... which has a history of its own to be overwritten
    other.restore(snap)
    moved = _chunks(other, x, b, 3, 6)
    assert np.array_equal(first, moved)
    assert m.counters()[4] == 0
    snap.free()
    a.close(); other.close(); m.destroy()


def test_snapshot_of_another_model_is_refused(dc):
    cfg = wl.tiny_flow()
    w = wl.make_workload(cfg)
    m1, m2 = dc.Model(cfg, w.weights), dc.Model(cfg, w.weights)
    s1, s2 = m1.open_stream(), m2.open_stream()
    snap = s1.snapshot()
    with pytest.raises(dc.DCError):
        s2.restore(snap)
    snap.free()
    s1.close(); s2.close(); m1.destroy(); m2.destroy()
