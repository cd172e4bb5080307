"""Edge cases of the GPU path against the oracle: maximum chunk length, a K/V cap shorter than a
chunk, a long K/V carry (many key blocks), batches larger than one slot table, single-frame chunks,
large dilations, a vocoder without residual blocks."""
import numpy as np
import pytest
import torch

import dc_workloads as wl
from oracle import dc_oracle as orc

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2
TOL_F32 = 1e-4


@pytest.fixture(scope="module")
def dc():
    import paper_2609_35115_b200 as dc
    dc.load_library()
    return dc


def _gu():
    from tests import gpu_util
    return gpu_util


def _check(dc, cfg, boundaries, tol):
    gu = _gu()
    w = wl.make_workload(cfg, boundaries=[boundaries])
    s = w.streams[0]
    ref = orc.run_stream(cfg, w.weights, s.feats, boundaries)
    m = dc.Model(cfg, w.weights)
    got = gu.run_gpu_stream(m, s.feats, boundaries)
    m.destroy()
    assert got.shape == ref.shape and np.isfinite(got).all()
    assert gu.rel_err(got, ref) <= tol, cfg.name


def test_flow_max_chunk_and_cap_shorter_than_chunk(dc):
    # f_chunk = 56 is the largest the slot layout admits; the carry keeps only 8 frames
    cfg = wl.tiny_flow(name="edge_cap8", hidden=128, n_heads=4, head_dim=32, kv_cap=8, f_chunk=56, mel_dim=16,
                       dilations=(4, 4), n_attn_layers=1, n_steps=2, seed=31)
    _check(dc, cfg, [0, 56, 57, 113, 120, 176, 177, 178, 234], TOL_BF16)


def test_flow_bulk_loader_small_ring_ragged(dc):
    # head_dim 64 without prompt rows takes the attention kernel's bulk-copy loader: a ring of 64 rows (cap 8 + chunk
    # 56) wraps inside almost every key block, the attended interval starts at every offset from its 8-row boundary
    # (single frames included), and the one key block is always partial (zero-filled V rows behind the last key)
    cfg = wl.tiny_flow(name="edge_bulk_cap8", hidden=128, n_heads=2, head_dim=64, kv_cap=8, f_chunk=56, mel_dim=16,
                       dilations=(2, 4), n_attn_layers=2, n_steps=2, seed=35)
    _check(dc, cfg, [0, 56, 57, 58, 61, 117, 120, 127, 183, 184, 191, 247, 250], TOL_BF16)
    # ... and a carry of 200 frames: two key blocks, the second one partial, interval offsets 0..7 by single-frame steps
    cfg = wl.tiny_flow(name="edge_bulk_cap200", hidden=64, n_heads=1, head_dim=64, kv_cap=200, f_chunk=50,
                       dilations=(1,), n_attn_layers=1, n_steps=1, seed=36)
    bnd = [0, 50, 100, 150, 200, 250] + [251 + i for i in range(9)] + [309, 359, 360, 410]
    _check(dc, cfg, bnd, TOL_BF16)


def test_flow_long_carry_many_key_blocks(dc):
    # kv_cap 700: up to 6 key blocks per query, ring of 750 rows wrapped once
    cfg = wl.tiny_flow(name="edge_cap700", hidden=64, n_heads=1, head_dim=64, kv_cap=700, f_chunk=50,
                       dilations=(1,), n_attn_layers=1, n_steps=1, seed=32)
    bnd = [0] + [50 * (i + 1) for i in range(17)] + [851, 880, 930]
    _check(dc, cfg, bnd, TOL_BF16)


def test_flow_single_frame_chunks(dc):
    cfg = wl.tiny_flow(name="edge_T1", n_steps=2, seed=33)
    _check(dc, cfg, list(range(0, 30)), TOL_BF16)


def test_flow_batch_larger_than_one_slot_table(dc):
    # 70 streams: two slot-table kernels, no captured graph for this batch size (direct launches)
    gu = _gu()
    cfg = wl.tiny_flow(name="edge_b70", n_streams=70, n_chunks=3, n_steps=2, seed=34)
    w = wl.make_workload(cfg)
    S = cfg.n_streams
    m = dc.Model(cfg, w.weights, max_batch=S)
    streams = [m.open_stream() for _ in range(S)]
    feats = [torch.from_numpy(s.feats).cuda() for s in w.streams]
    outs = [torch.empty(s.feats.shape[0], cfg.mel_dim, device="cuda") for s in w.streams]
    for r in range(cfg.n_chunks):
        fs = [feats[i][w.streams[i].boundaries[r]:w.streams[i].boundaries[r + 1]] for i in range(S)]
        os_ = [outs[i][w.streams[i].boundaries[r]:w.streams[i].boundaries[r + 1]] for i in range(S)]
        dc.decode_batch(m, streams, fs, os_)
    torch.cuda.synchronize()
    assert m.counters()[4] == 0
    for i in (0, 1, 63, 64, 69):
        si = w.streams[i]
        ref = orc.run_stream(cfg, w.weights, si.feats, si.boundaries)
        assert gu.rel_err(outs[i].cpu().numpy(), ref) <= TOL_BF16
    # a subset of the streams in another order is a valid batch, too
    sub = [5, 2, 66]
    more = [torch.from_numpy(np.random.default_rng(9).standard_normal((4, cfg.in_dim), dtype=np.float32)).cuda() for _ in sub]
    o2 = [torch.empty(4, cfg.mel_dim, device="cuda") for _ in sub]
    dc.decode_batch(m, [streams[i] for i in sub], more, o2)
    torch.cuda.synchronize()
    assert all(torch.isfinite(o).all() for o in o2) and m.counters()[4] == 0
    for st in streams:
        st.close()
    m.destroy()


def test_conv_stream_large_dilation(dc):
    cfg = wl.CONFIGS["cfg1"].replace(name="edge_d64", hidden=16, dilations=(64, 1), f_chunk=24, seed=35, bias_std=0.2)
    _check(dc, cfg, [0, 24, 25, 49, 73, 80, 104, 128, 152, 176, 200], TOL_F32)


def test_vocoder_without_residual_blocks_and_big_stride(dc):
    cfg = wl.tiny_vocoder(name="edge_voc", up_strides=(16,), up_channels=(8, 12), res_dilations=(), f_chunk=7, seed=36)
    _check(dc, cfg, [0, 7, 8, 15, 16, 23], TOL_F32)


def test_misaligned_device_pointers_are_refused_before_any_launch(dc):
    """The kernels access the caller's chunk, output and weights with 16-byte loads and stores; a pointer
    that is not 16-byte aligned is refused with DC_ERR_ARG before anything is launched (the check is on
    the host, so nothing here reaches the device), and the stream stays usable and untouched."""
    lib = dc.load_library()
    for cfg in (wl.CONFIGS["cfg1"], wl.tiny_flow(), wl.tiny_vocoder()):
        w = wl.make_workload(cfg)
        s = w.streams[0]
        m = dc.Model(cfg, w.weights, max_batch=cfg.n_steps if cfg.pipeline == "flow" else 1)
        st = m.open_stream()
        T = s.boundaries[1]
        x = torch.from_numpy(s.feats[:T]).cuda()
        y = torch.zeros(T * cfg.out_per_frame + 8, device="cuda")
        before = m.counters()
        assert st.decode_raw(x.data_ptr() + 4, T - 1, y.data_ptr()) == 1
        assert "16-byte aligned" in lib.dc_last_error().decode()
        assert st.decode_raw(x.data_ptr(), T, y.data_ptr() + 8) == 1
        after = m.counters()
        assert after[3] == before[3] + 2 and after[5] == before[5] and after[0] == before[0]
        if cfg.pipeline == "flow":
            with pytest.raises(dc.DCError):
                dc.decode_batch(m, [st], [x.view(-1)[1:1 + (T - 1) * cfg.in_dim].view(T - 1, cfg.in_dim)],
                                [y[:(T - 1) * cfg.out_per_frame].view(T - 1, -1)])
            with pytest.raises(dc.DCError):
                dc.decode_wavefront_batch(m, [st], [x], [y[1:1 + T * cfg.out_per_frame]])
            assert m.counters()[5] == before[5]
        # the refused calls left the stream as it was: the chunk decodes as the first chunk of a fresh stream
        got = st.decode_chunk(x).clone().reshape(-1).cpu().numpy()
        ref = orc.run_stream(cfg, w.weights, s.feats[:T], [0, T]).reshape(-1)
        assert _gu().rel_err(got, ref) <= (TOL_F32 if cfg.precision == "f32" else TOL_BF16)
        st.close()
        m.destroy()
    # the allocation-free entry point checks its three device pointers the same way
    C = 64
    wts = torch.zeros(3 * C * C + C + 4, device="cuda")
    xs = torch.zeros(8 * C + 4, device="cuda")
    ys = torch.zeros(8 * C + 4, device="cuda")
    assert dc.conv_stack_noalloc(wts[1:], C, (1,), xs[:8 * C].view(8, C), ys[:8 * C].view(8, C)) == 1
    assert "16-byte aligned" in lib.dc_last_error().decode()
    assert dc.conv_stack_noalloc(wts, C, (1,), xs[1:1 + 8 * C].view(8, C), ys[:8 * C].view(8, C)) == 1
    assert dc.conv_stack_noalloc(wts, C, (1,), xs[:8 * C].view(8, C), ys[3:3 + 8 * C].view(8, C)) == 1
    assert dc.conv_stack_noalloc(wts, C, (1,), xs[:8 * C].view(8, C), ys[:8 * C].view(8, C)) == 0
    torch.cuda.synchronize()


def test_host_entry_point_stages_a_misaligned_pinned_buffer(dc):
    """A page-locked host buffer at an odd float offset cannot be read by the kernels directly; the host
    entry points fall back to their staging copy and give the same bytes."""
    cfg = wl.tiny_flow()
    w = wl.make_workload(cfg)
    s = w.streams[0]
    T = s.boundaries[1]
    m = dc.Model(cfg, w.weights)
    pin_in = torch.zeros(T * cfg.in_dim + 4).pin_memory()
    pin_out = torch.zeros(T * cfg.mel_dim + 4).pin_memory()
    outs = []
    for off in (0, 1):
        st = m.open_stream()
        fi = pin_in[off:off + T * cfg.in_dim].view(T, cfg.in_dim)
        fo = pin_out[off:off + T * cfg.mel_dim].view(T, cfg.mel_dim)
        fi.copy_(torch.from_numpy(s.feats[:T]))
        assert st.decode_chunk_host(fi, fo) == T * cfg.mel_dim
        outs.append(fo.clone().numpy())
        st.close()
    m.destroy()
    assert np.array_equal(outs[0], outs[1])
