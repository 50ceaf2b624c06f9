"""Layer stacks: several fully-connected layers in one call, with the relay kernel between staged layers."""
import numpy as np
import pytest
import torch

import oracle
import paper_1708_08917_b200 as circ
from paper_1708_08917_b200 import synth
from gpu_helpers import TOL_F32, scale_rel_err

pytestmark = pytest.mark.gpu


def make_layers(name, dims, ks, relu_last=False, bias=True):
    """dims = [n0, n1, ..., nD]; layer l maps dims[l] -> dims[l+1] with block size ks[l]."""
    specs = []
    for l in range(len(dims) - 1):
        n, m, k = dims[l], dims[l + 1], ks[l]
        w = synth.normal((m // k, n // k, k), 2.0 / n, synth.stream_id(name, f"w{l}"))
        b = synth.normal((m,), 0.01, synth.stream_id(name, f"b{l}")) if bias else None
        specs.append((m, n, k, w, b, relu_last or l + 2 < len(dims)))
    return specs


def oracle_stack(specs, x, convention=0):
    a = x
    for (m, n, k, w, b, relu) in specs:
        a = oracle.fc(w, a, bias=b, relu=relu, convention=convention)
    return a


def run_stack(specs, x, variants=None, convention=0, reserve=False):
    handles = []
    s = None
    try:
        for l, (m, n, k, w, b, relu) in enumerate(specs):
            h = circ.circ_fc_create(m, n, k, w)
            handles.append(h)
            if b is not None:
                circ.circ_set_bias(h, b)
            circ.circ_set_activation(h, int(relu))
            circ.circ_set_convention(h, convention)
            if variants:
                circ.circ_set_variant(h, variants[l])
        s = circ.circ_stack_create(handles)
        batch = x.shape[0]
        if reserve:
            circ.circ_stack_reserve(s, batch)
        xd = torch.from_numpy(x).cuda()
        y = torch.full((batch, specs[-1][0]), float("nan"), device="cuda")
        circ.circ_stack_forward(s, xd, y, batch, torch.cuda.current_stream())
        torch.cuda.synchronize()
        for h in handles:
            circ.circ_device_status(h)
        # layer by layer through the ordinary forward, for comparison
        a = xd
        for h, (m, n, k, w, b, relu) in zip(handles, specs):
            o = torch.empty(batch, m, device="cuda")
            circ.circ_fc_forward(h, a, o, batch)
            a = o
        torch.cuda.synchronize()
        return (y.cpu().numpy().astype(np.float64), a.cpu().numpy().astype(np.float64), circ.circ_stack_relayed(s),
                [circ.circ_last_variant(h) for h in handles])
    finally:
        circ.circ_stack_destroy(s)
        for h in handles:
            circ.circ_destroy(h)


T, F, A = circ.CIRC_VARIANT_TENSOR, circ.CIRC_VARIANT_STAGED, circ.CIRC_VARIANT_AUTO


@pytest.mark.parametrize("dims,ks,batch,variants,relayed", [
    ([512, 256, 256, 128], [16, 16, 16], 40, None, 2),            # all tensor path
    ([512, 256, 256, 128], [16, 16, 16], 33, None, 2),            # odd batch: the last pair has one sample
    ([256, 384, 128], [32, 32], 9, [F, F], 1),                    # float32 FMA contraction on both sides
    ([256, 512, 256, 64], [32, 32, 32], 64, [T, F, T], 2),        # relay into either operand format
    ([96, 48, 80], [16, 16], 50, None, 1),                        # q, p not multiples of 4 or 8: scalar gather / scatter
    ([512, 256, 256], [16, 32], 40, None, 0),                     # block size changes: through the activation buffer
    ([512, 256, 128], [16, 16], 4, None, 0),                      # small batch: single-launch kernels
    ([1024, 512], [64], 20, None, 0),                             # a stack of one
    ([2048, 1024, 1024, 512, 256], [4, 4, 4, 4], 300, None, 3),   # k = 4, several column tiles
    ([1024, 1024, 512], [256, 256], 70, None, 1),                 # k = 256
])
def test_stack_matches_oracle_chain(dims, ks, batch, variants, relayed):
    name = f"stack_{'_'.join(map(str, dims))}_{batch}"
    specs = make_layers(name, dims, ks)
    x = synth.normal((batch, dims[0]), 1.0, synth.stream_id(name, "x"), absolute=True)
    got, layerwise, n_relayed, used = run_stack(specs, x, variants)
    ref = oracle_stack(specs, x)
    assert not np.isnan(got).any()
    assert n_relayed == relayed
    assert scale_rel_err(got, ref) <= TOL_F32
    assert scale_rel_err(got, layerwise) <= TOL_F32
    if variants:
        assert used == variants


def test_stack_convention_1_and_reserve():
    dims, ks, batch = [256, 256, 128], [16, 16], 24
    specs = make_layers("stack_conv1", dims, ks)
    x = synth.normal((batch, dims[0]), 1.0, synth.stream_id("stack_conv1", "x"))
    got, _, n_relayed, _ = run_stack(specs, x, convention=1, reserve=True)
    assert n_relayed == 1
    assert scale_rel_err(got, oracle_stack(specs, x, convention=1)) <= TOL_F32


def test_config3_stack_in_one_call():
    # 9216 -> 4096 -> 4096 -> 1024, k = 128, batch 128, ReLU between layers; the oracle chains the three layers on sampled rows
    layers = synth.config3_layers(128)
    specs = [(c.m, c.n, c.k, c.w, None, c.relu) for c in layers]
    x = layers[0].x
    got, layerwise, n_relayed, used = run_stack(specs, x)
    assert n_relayed == 2 and used == [T, T, T]
    rows = [0, 63, 64, 127]
    assert scale_rel_err(got[rows], oracle_stack(specs, x[rows])) <= TOL_F32
    assert scale_rel_err(got, layerwise) <= TOL_F32


def test_stack_in_a_cuda_graph():
    dims, ks, batch = [512, 256, 128], [16, 16], 32
    specs = make_layers("stack_graph", dims, ks)
    x = synth.normal((batch, dims[0]), 1.0, synth.stream_id("stack_graph", "x"))
    handles = [circ.circ_fc_create(m, n, k, w) for (m, n, k, w, b, relu) in specs]
    s = circ.circ_stack_create(handles)
    try:
        circ.circ_stack_reserve(s, batch)
        xd = torch.from_numpy(x).cuda()
        y = torch.zeros(batch, dims[-1], device="cuda")
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            circ.circ_stack_forward(s, xd, y, batch, torch.cuda.current_stream())
        y.zero_()
        g.replay()
        torch.cuda.synchronize()
        ref = oracle_stack([(m, n, k, w, None, False) for (m, n, k, w, b, relu) in specs], x)
        assert scale_rel_err(y.cpu().numpy().astype(np.float64), ref) <= TOL_F32
    finally:
        circ.circ_stack_destroy(s)
        for h in handles:
            circ.circ_destroy(h)


def test_stack_rejects_bad_arguments():
    w = synth.normal((2, 2, 16), 1.0, 5)
    a = circ.circ_fc_create(32, 32, 16, w)
    b = circ.circ_fc_create(32, 64, 16, synth.normal((2, 4, 16), 1.0, 6))
    c = circ.circ_conv_create(16, 16, 3, 1, 16, synth.normal((3, 3, 1, 1, 16), 1.0, 7))
    try:
        with pytest.raises(circ.CircError) as e:
            circ.circ_stack_create([a, b])        # 32 outputs into 64 inputs
        assert e.value.code == circ.CIRC_ERR_SHAPE
        with pytest.raises(circ.CircError) as e:
            circ.circ_stack_create([a, c])
        assert e.value.code == circ.CIRC_ERR_ARG
        with pytest.raises(circ.CircError) as e:
            circ.circ_stack_create([])
        assert e.value.code == circ.CIRC_ERR_ARG
        s = circ.circ_stack_create([b, a])
        x = torch.zeros(4, 64, device="cuda")
        y = torch.zeros(4, 32, device="cuda")
        with pytest.raises(circ.CircError) as e:
            circ.circ_stack_forward(s, x, y, 0)
        assert e.value.code == circ.CIRC_ERR_SHAPE
        with pytest.raises(circ.CircError) as e:
            circ.circ_stack_forward(s, x, None, 4)
        assert e.value.code == circ.CIRC_ERR_ARG
        circ.circ_stack_destroy(s)
    finally:
        for h in (a, b, c):
            circ.circ_destroy(h)
