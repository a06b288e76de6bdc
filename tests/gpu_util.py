"""Helpers of the GPU parity tests: one context per session, numpy <-> device copies."""
import numpy as np
import torch

_ctx = None


def ctx():
    global _ctx
    if _ctx is None:
        from paper_2101_01321_b200 import build, binding
        build.build()
        _ctx = binding.Context(0)
    return _ctx


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def host(t):
    return t.cpu().numpy()


def assert_same(got, want, what=""):
    got = np.asarray(got)
    want = np.asarray(want)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    bad = np.flatnonzero(got.reshape(-1) != want.reshape(-1))
    assert bad.size == 0, (f"{what}: {bad.size} of {got.size} differ; first at {bad[:5]}: "
                           f"got {got.reshape(-1)[bad[:5]]}, want {want.reshape(-1)[bad[:5]]}")
