"""Helpers of the GPU parity tests: run a workload through the C-ABI library."""
import numpy as np
import torch

import paper_2609_35115_b200 as dc


def run_gpu_stream(model, feats: np.ndarray, boundaries, stream=None) -> np.ndarray:
    """Feeds one stream chunk by chunk through dc_decode_chunk; returns the concatenated output."""
    st = stream or model.open_stream()
    x = torch.from_numpy(np.ascontiguousarray(feats)).cuda()
    outs = []
    cfg = model.cfg
    la = getattr(cfg, "f_lookahead", 0)       # a full call also presents the next <= la frames (not committed)
    for c in range(len(boundaries) - 1):
        lo, hi = boundaries[c], boundaries[c + 1]
        if la and hi - lo == cfg.f_chunk:
            hi = min(hi + la, boundaries[-1])
        outs.append(st.decode_chunk(x[lo:hi].contiguous()).clone())
    torch.cuda.synchronize()
    assert model.counters()[4] == 0, "a bounded device-side wait timed out"
    if stream is None:
        st.close()
    return torch.cat([o.reshape(-1) if o.dim() == 1 else o for o in outs], dim=0).cpu().numpy()


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """max |err| / RMS(ref) over all output elements of the stream's run."""
    ref = ref.astype(np.float64)
    return float(np.abs(got.astype(np.float64) - ref).max() / np.sqrt((ref ** 2).mean()))
