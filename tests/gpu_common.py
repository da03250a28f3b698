"""Helpers shared by the GPU parity tests: run the CUDA library and the CPU oracle on the same
seeded inputs and compare byte for byte."""
import numpy as np

import oracle
from paper_2207_07736_b200 import binding


def torch_cuda():
    import torch
    assert torch.cuda.is_available(), "GPU test needs a CUDA device"
    return torch


def to_np(t):
    return None if t is None else t.cpu().numpy()


def assert_same_bits(a, b, what):
    a, b = np.ascontiguousarray(a), np.ascontiguousarray(b)
    assert a.shape == b.shape and a.dtype == b.dtype, (what, a.shape, b.shape, a.dtype, b.dtype)
    if not np.array_equal(a.view(np.uint8), b.view(np.uint8)):
        av = a.reshape(-1).view(np.uint32 if a.dtype.itemsize == 4 else np.uint8)
        bv = b.reshape(-1).view(av.dtype)
        bad = np.flatnonzero(av != bv)
        idx = np.unravel_index(bad[0] * (1 if a.dtype.itemsize in (1, 4) else 1), a.shape) if a.dtype.itemsize in (1, 4) else bad[0]
        raise AssertionError("%s differs in %d of %d elements; first at %s: gpu=%r oracle=%r" % (
            what, bad.size, av.size, idx, a.reshape(-1)[bad[0]], b.reshape(-1)[bad[0]]))


def compare_rollout(gpu_out, sim, orc_out, orc, env_ids=None, what=""):
    """gpu_out: dict of torch tensors [T,N,...]; orc_out: oracle dict over env_ids (default all)."""
    sel = slice(None) if env_ids is None else np.asarray(env_ids, dtype=np.int64)
    for k in ("obs", "act", "rew", "done"):
        if gpu_out.get(k) is None:
            continue
        g = to_np(gpu_out[k])[:, sel]
        assert_same_bits(g, orc_out[k], "%s %s" % (what, k))
    st = to_np(sim.state())[sel]
    ep, rc, t = sim.counters()
    assert_same_bits(st, orc.state, what + " final state")
    assert_same_bits(to_np(ep)[sel].astype(np.uint32), orc.ep_len, what + " ep_len")
    assert_same_bits(to_np(rc)[sel].astype(np.uint32), orc.reset_count, what + " reset_count")
    assert t == orc.t, (what, t, orc.t)
