"""Repeated forward passes give identical bits: a race between the roles of a kernel (TMA producer,
MMA issuer, epilogue warps, cluster peers) or between consecutive launches overlapped by programmatic
stream serialization would show up as a run-to-run difference.  Small batches take the split-K GEMM,
the row-sharing attention and the two-kernel linear + LayerNorm; the larger one the cluster kernel."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import assert_same, ctx, dev, host
from paper_2101_01321_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,layers,repeats", [(1, 3, 40), (8, 2, 25), (40, 2, 10)])
def test_layer_stack_is_repeatable(B, layers, repeats):
    L = 128
    x, params = synth.make_model(2, B, layers=layers)
    c = ctx()
    objs = [c.ibert_layer_create(p) for p in params]
    xd = dev(x)
    first = None
    for _ in range(repeats):
        h = xd
        for ly in objs:
            h, _ = c.ibert_encoder_layer(ly, h, B, L)
        got = host(h)
        if first is None:
            first = got
        else:
            assert_same(got, first, "repeat of the layer stack")
    c.check()
    for ly in objs:
        ly.close()
    if B <= 8:                                     # and the bits are the oracle's
        h = x
        for p in params:
            h = oracle.encoder_layer(p, h, B, L).out
        assert_same(first, h, "layer stack vs oracle")
