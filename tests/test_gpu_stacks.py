"""GPU parity on the ResNet-18- and VGG-16-shaped convolution stacks.

* full-size layers (batch 256 / 64): every distinct layer shape on its own seeded input; packed planes,
  int32 accumulators and fp32 outputs are compared with the oracle IN FULL, a group of images at a time.
  The oracle's naive convolution needs seconds to tens of seconds per layer on the host cores; should a
  slow host exceed FULL_COMPARE_BUDGET_S for one layer, the images not reached by then are compared on
  sampled outputs (complete rows plus random entries) and the test prints which route each layer took;
* the whole stack chained at batch 2: each side feeds its own previous output forward (ReLU fused into
  the next encode, 2x2 max-pool by the harness), every layer's accumulators and outputs compared in full.
"""
import time

import numpy as np
import pytest

import oracle
from helpers import assert_fp32_close, oracle_weight_planes
from paper_2106_09886_b200 import workloads as wl

pytestmark = pytest.mark.gpu

FULL_COMPARE_BUDGET_S = 150.0     # per layer; the oracle needs 2-30 s per layer on a 16-core host


def distinct(shapes):
    seen, out = set(), []
    for i, s in enumerate(shapes):
        key = (s.H, s.W, s.C, s.Cout, s.R, s.stride)
        if key not in seen:
            seen.add(key)
            out.append((i, s))
    return out


RESNET = distinct(wl.resnet18_shapes())
VGG = distinct(wl.vgg16_shapes())


def run_full_size_layer(config, li, s):
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    a = wl.layer_input(0, config, li, s, signed=(s.C == 3))
    w = wl.he_weights(0, config, li, s)
    sa, sw = wl.per_tensor_scale(a, s.ab), wl.per_tensor_scale(w, s.wb)
    alpha = np.float32(sa * sw)
    relu = s.C != 3
    qa = oracle.quantize(a, s.ab, sa, relu)
    qw = oracle.quantize(w, s.wb, sw)
    a_d = torch.from_numpy(a).to(dev)
    planes = qnn.encode_pack(a_d.view(-1, s.C), s.ab, sa, qnn.RELU if relu else 0)
    del a_d
    packed = qnn.pack_weights(torch.from_numpy(w).to(dev), s.Cout, s.R * s.S, s.C, qnn.W_NTC, s.wb, sw)
    out, acc = qnn.bconv2d(planes, s.ab, packed, s.wb, s.N, s.H, s.W, s.C, s.Cout, s.R, s.S, s.stride, s.pad, alpha,
                           want_acc=True)
    torch.cuda.synchronize()
    # packed planes in full
    assert np.array_equal(planes.cpu().numpy().view(np.uint32), oracle.pack_planes(qa.reshape(-1, s.C), s.ab))
    wp, ts = qnn.weights_views(packed, s.Cout, s.R * s.S, s.C, s.wb)
    want_wp, want_ts = oracle_weight_planes(qw.reshape(s.Cout, s.R * s.S, s.C), s.wb)
    assert np.array_equal(wp.cpu().numpy().view(np.uint32), want_wp) and np.array_equal(ts.cpu().numpy(), want_ts)
    del planes
    acc_h = acc.cpu().numpy().reshape(s.N, -1, s.Cout)
    out_h = out.cpu().numpy().reshape(s.N, -1, s.Cout)
    del acc, out
    # every accumulator and output, a group of images at a time (a convolution is independent per image)
    group = max(1, s.N // 16)
    t0, n_done = time.perf_counter(), 0
    while n_done < s.N and time.perf_counter() - t0 < FULL_COMPARE_BUDGET_S:
        n1 = min(s.N, n_done + group)
        want = oracle.conv2d(qa[n_done:n1], qw, s.stride, s.pad).reshape(n1 - n_done, -1, s.Cout)
        assert np.array_equal(acc_h[n_done:n1], want), f"{s.name}: accumulators differ in images {n_done}..{n1 - 1}"
        assert_fp32_close(out_h[n_done:n1], oracle.scale(want, alpha))
        n_done = n1
    route = "full"
    if n_done < s.N:
        # host too slow for the budget: the remaining images on sampled outputs (full rows + random entries)
        route = f"full for images 0..{n_done - 1}, sampled for the rest"
        rest = s.N - n_done
        rows, cols = wl.sample_pairs(li, rest * s.Ho * s.Wo, s.Cout, 60000, full_rows=40)
        want = oracle.conv2d_sampled(qa[n_done:], qw, s.stride, s.pad, rows, cols)
        assert np.array_equal(acc_h[n_done:].reshape(-1, s.Cout)[rows, cols], want)
        assert_fp32_close(out_h[n_done:].reshape(-1, s.Cout)[rows, cols], oracle.scale(want, alpha))
        assert np.array_equal(out_h[n_done:], oracle.scale(acc_h[n_done:], alpha))
    print(f"[stacks] {s.name}: compared {route} ({time.perf_counter() - t0:.1f} s of oracle time)")


@pytest.mark.parametrize("li,s", RESNET, ids=[s.name for _, s in RESNET])
def test_resnet18_layers_full_size(li, s):
    run_full_size_layer(4, li, s)


@pytest.mark.parametrize("li,s", VGG, ids=[s.name for _, s in VGG])
def test_vgg16_layers_full_size(li, s):
    run_full_size_layer(5, li, s)


def chain(shapes, config, first_signed):
    import torch
    from paper_2106_09886_b200 import qnn
    dev = torch.device("cuda:0")
    s0 = shapes[0]
    x_o = wl.layer_input(0, config, 100, s0, signed=first_signed)      # oracle-side activation
    x_g = torch.from_numpy(x_o).to(dev)                                 # library-side activation
    first = True
    for li, s in enumerate(shapes):
        assert x_o.shape == (s.N, s.H, s.W, s.C)
        w = wl.he_weights(0, config, li, s)
        relu = not (first and first_signed)
        x_act = np.maximum(x_o, 0) if relu else x_o                     # range of what the encoder sees
        sa, sw = wl.per_tensor_scale(x_act, s.ab), wl.per_tensor_scale(w, s.wb)
        absmax = qnn.absmax_f32(x_g.clamp(min=0).contiguous() if relu else x_g)
        assert np.float32(absmax.cpu().numpy()[0]) == np.float32(np.abs(x_act).max())
        alpha = np.float32(sa * sw)
        qa = oracle.quantize(x_o, s.ab, sa, relu)
        qw = oracle.quantize(w, s.wb, sw)
        acc_o = oracle.conv2d(qa, qw, s.stride, s.pad)
        out_o = oracle.scale(acc_o, alpha)
        planes = qnn.encode_pack(x_g.view(-1, s.C), s.ab, sa, qnn.RELU if relu else 0)
        packed = qnn.pack_weights(torch.from_numpy(w).to(dev), s.Cout, s.R * s.S, s.C, qnn.W_NTC, s.wb, sw)
        out_g, acc_g = qnn.bconv2d(planes, s.ab, packed, s.wb, s.N, s.H, s.W, s.C, s.Cout, s.R, s.S, s.stride, s.pad,
                                   alpha, want_acc=True)
        torch.cuda.synchronize()
        assert np.array_equal(acc_g.cpu().numpy(), acc_o), s.name
        assert_fp32_close(out_g.cpu().numpy(), out_o)
        if s.branch:
            continue                      # 1x1 projection: evaluated on its stage's input, not fed forward
        x_o, x_g = out_o, out_g
        if s.pool_after:
            x_o = wl.maxpool2x2_nhwc(np.maximum(x_o, 0))                # pool after ReLU; ReLU again is a no-op
            x_g = torch.nn.functional.max_pool2d(x_g.clamp(min=0).permute(0, 3, 1, 2), 2).permute(0, 2, 3, 1).contiguous()
            assert np.array_equal(x_g.cpu().numpy(), x_o)
        first = False


def reorder_branches(shapes):
    """Put each 1x1 projection before the 3x3 convolution that shares its input."""
    out = []
    for s in shapes:
        if s.branch:
            out.insert(len(out) - 1, s)
        else:
            out.append(s)
    return out


def test_resnet18_stack_chained_batch2():
    chain(reorder_branches(wl.resnet18_shapes(batch=2)), 4, first_signed=False)


def test_vgg16_stack_chained_batch2():
    chain(wl.vgg16_shapes(batch=2), 5, first_signed=True)


@pytest.mark.parametrize("precision", [1, 2])
def test_resnet18_mixed_precision_chained_batch2(precision):
    """Table 4's mixed precisions (8x8, 8x7, 8x6 / 4x5, 4x3, 4x2 bits per stage), whole stack chained at batch 2."""
    chain(reorder_branches(wl.resnet18_mixed_shapes(precision, batch=2)), 40 + precision, first_signed=False)
