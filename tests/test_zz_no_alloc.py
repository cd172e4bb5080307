"""dc_conv_stack_noalloc: the entry point for callers that cannot allocate device memory (a fixed
memory budget, a foreign allocator's pool, a real-time audio callback).  It must give what the
ordinary stream API gives for the same network and input - and what the CPU oracle's offline run
over the whole sequence gives - call after call, although every call shares one built-in scratch
array that still holds the previous call's values.

Collected last on purpose: if it fails, a run that stops at the first failure has already run
every other test."""
import numpy as np
import pytest
import torch

import dc_workloads as wl
from oracle import dc_oracle as orc

pytestmark = pytest.mark.gpu

TOL_F32 = 1e-4


def _stream_api_result(dc, cfg, weights, x):
    """The existing entry points: dc_create + dc_stream_open + dc_decode_chunk, chunk by chunk."""
    m = dc.Model(cfg, weights)
    st = m.open_stream()
    xd = torch.from_numpy(x).cuda()
    outs = [st.decode_chunk(xd[lo:lo + cfg.f_chunk].contiguous()).clone() for lo in range(0, x.shape[0], cfg.f_chunk)]
    torch.cuda.synchronize()
    st.close()
    m.destroy()
    return torch.cat(outs).cpu().numpy()


def _rel_err(got, ref):
    return float(np.abs(got.astype(np.float64) - ref).max() / np.sqrt((ref.astype(np.float64) ** 2).mean()))


def test_noalloc_entry_matches_stream_api_on_two_calls_in_a_row():
    import paper_2609_35115_b200 as dc
    dc.load_library()
    rng = np.random.default_rng(77)
    # call 1: long sequence, small dilations; call 2: shorter sequence, larger dilation, other
    # weights - whatever call 1 left in the shared array must not leak into call 2
    cases = [
        (wl.CONFIGS["cfg1"].replace(name="na1", dilations=(1, 2, 1), f_chunk=16, bias_std=0.2, seed=5), 200),
        (wl.CONFIGS["cfg1"].replace(name="na2", dilations=(4, 1), f_chunk=16, bias_std=0.2, seed=6), 37),
    ]
    prepared = []
    for cfg, n_frames in cases:
        weights = wl.make_weights(cfg, np.random.default_rng(cfg.seed))
        x = rng.standard_normal((n_frames, cfg.hidden), dtype=np.float32)
        ref = _stream_api_result(dc, cfg, weights, x)
        # the existing entry point itself against the oracle's definition (offline causal run)
        assert _rel_err(ref, orc.conv_stack_offline(cfg, weights, x)) <= TOL_F32, cfg.name
        prepared.append((cfg, weights, x, ref))
    # everything the new entry point touches is allocated here, by the caller, beforehand
    bufs = [(torch.from_numpy(w).cuda(), torch.from_numpy(x).cuda(), torch.full(x.shape, 7.0, device="cuda"))
            for _, w, x, _ in prepared]
    torch.cuda.synchronize()
    for (cfg, _, _, ref), (wd, xd, yd) in zip(prepared, bufs):
        assert dc.conv_stack_noalloc(wd, cfg.hidden, cfg.dilations, xd, yd) == 0
    torch.cuda.synchronize()
    for (cfg, weights, x, ref), (_, _, yd) in zip(prepared, bufs):
        got = yd.cpu().numpy()
        assert got.shape == ref.shape
        assert _rel_err(got, ref) <= TOL_F32, cfg.name
        assert _rel_err(got, orc.conv_stack_offline(cfg, weights, x)) <= TOL_F32, cfg.name
    # the same two calls again, in the other order, still agree
    for (cfg, _, _, ref), (wd, xd, yd) in reversed(list(zip(prepared, bufs))):
        yd.fill_(-3.0)
        assert dc.conv_stack_noalloc(wd, cfg.hidden, cfg.dilations, xd, yd) == 0
        torch.cuda.synchronize()
        assert _rel_err(yd.cpu().numpy(), ref) <= TOL_F32, cfg.name


def test_noalloc_entry_refuses_sizes_beyond_its_scratch():
    import paper_2609_35115_b200 as dc
    lib = dc.load_library()
    C = 64
    w = torch.zeros(3 * C * C + C, device="cuda")
    n_big = dc.NOALLOC_SCRATCH_FLOATS // (2 * C)          # P = n_big would fit, but n_big + halo rounds up to 2P
    x = torch.zeros(n_big, C, device="cuda")
    y = torch.zeros(n_big, C, device="cuda")
    assert dc.conv_stack_noalloc(w, C, (1,), x, y) == 1    # DC_ERR_ARG
    msg = lib.dc_last_error().decode()
    assert "scratch floats" in msg and str(dc.NOALLOC_SCRATCH_FLOATS) in msg
    assert dc.conv_stack_noalloc(w, C, (1,), x[: n_big - 2], y[: n_big - 2]) == 0   # exactly at the limit
    assert dc.conv_stack_noalloc(w, 62, (1,), x, y) == 1
    torch.cuda.synchronize()
