"""A stack of encoder layers captured into a CUDA graph gives the same bytes as the eager calls,
on every replay and for new contents of its input buffer."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import assert_same, dev, host
from paper_2101_01321_b200 import binding, build, synth

pytestmark = pytest.mark.gpu

_own = None


def ctx():
    """A context on a stream of its own: the default stream cannot be captured."""
    global _own
    if _own is None:
        build.build()
        _own = binding.Context(0, torch.cuda.Stream())
    return _own


@pytest.mark.parametrize("B,L,H,heads,F,masked", [(2, 64, 256, 4, 512, False), (3, 100, 128, 2, 256, True),
                                                  (1, 128, 768, 12, 3072, False)])
def test_graph_replay_equals_eager_and_oracle(B, L, H, heads, F, masked):
    x, params = synth.make_model(0, B, layers=3, H=H, heads=heads, F=F, L=L)
    lens = np.array([L, max(L // 3, 1), 1][:B], np.int32) if masked else None
    c = ctx()
    layers = [c.ibert_layer_create(p) for p in params]
    x_d = dev(x)
    out_d = torch.empty((B * L, H), dtype=torch.int8, device="cuda")
    lens_d = dev(lens) if masked else None
    torch.cuda.synchronize()
    g = binding.Graph(c, layers, x_d, B, L, out_d, lens_d)
    want = x
    for p in params:
        want = oracle.encoder_layer(p, want, B, L, lens=lens).out
    for _ in range(3):
        out_d.zero_()
        torch.cuda.synchronize()            # the buffers are prepared on the default stream
        g.launch()
        c.check()
        assert_same(host(out_d), want, "graph replay")
    # new contents in the same input buffer
    x2 = np.roll(x, 7, axis=0).copy()
    x_d.copy_(dev(x2))
    torch.cuda.synchronize()
    g.launch()
    c.check()
    want2 = x2
    for p in params:
        want2 = oracle.encoder_layer(p, want2, B, L, lens=lens).out
    assert_same(host(out_d), want2, "graph replay, new input")
    # the eager path still works beside the graph (its workspace is its own)
    h = x_d
    for ly in layers:
        h, _ = (c.ibert_encoder_layer_masked(ly, h, B, L, lens_d) if masked else c.ibert_encoder_layer(ly, h, B, L))
    c.check()
    assert_same(host(h), want2, "eager beside graph")
    g.close()
    for ly in layers:
        ly.close()


def test_graph_creation_rejects_profiling_and_bad_arguments():
    x, params = synth.make_model(0, 1, layers=1, H=128, heads=2, F=256, L=16)
    c = ctx()
    layer = c.ibert_layer_create(params[0])
    x_d = dev(x)
    out_d = torch.empty((16, 128), dtype=torch.int8, device="cuda")
    c.ibert_profile_begin()
    with pytest.raises(binding.IbertError):
        binding.Graph(c, [layer], x_d, 1, 16, out_d)
    c.ibert_profile_end()
    with pytest.raises(binding.IbertError):
        binding.Graph(c, [layer], x_d, 1, 1000, out_d)          # L out of range
    g = binding.Graph(c, [layer], x_d, 1, 16, out_d)
    g.launch()
    c.check()
    assert_same(host(out_d), oracle.encoder_layer(params[0], x, 1, 16).out, "single-layer graph")
    g.close()
    layer.close()
    # a context on the default stream cannot capture
    from gpu_util import ctx as default_ctx
    d = default_ctx()
    layer_d = d.ibert_layer_create(params[0])
    with pytest.raises(binding.IbertError):
        binding.Graph(d, [layer_d], x_d, 1, 16, out_d)
    layer_d.close()
