"""GPU parity of whole layer stacks against the oracle: every code tensor of
every layer bit-exact at a batch the oracle finishes in seconds, and sampled
images of the full-size batch the benchmark times."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from oracle import native, stack as ostack
import dsq_inputs
from gpu_util import T, N


@pytest.fixture(scope="module")
def dsq():
    import paper_1908_05033_b200 as d
    return d


def compare_stack(st, wid, batch, w_offset=0.5, debug=True):
    from paper_1908_05033_b200.stack import GpuStack
    x = dsq_inputs.stack_input(st, batch=batch, workload_id=wid)
    params = dsq_inputs.stack_params(st, workload_id=wid)
    ref = ostack.run_stack(st, x, params, w_offset=w_offset)
    g = GpuStack(st, params, batch=batch, w_offset=w_offset, keep_debug=debug)
    g.forward(T(x))
    g.check()
    for name in st.tensor_shapes():
        got = N(g.unpack(name))
        assert np.array_equal(got, ref[name]), name
        # padding lanes of every packed tensor are zero
        H, W, Cc = g.shapes[name]
        packed = N(g.codes[name]).reshape(-1, g.codes[name].shape[-1])
        assert np.array_equal(
            packed, native.pack_rows(ref[name].reshape(-1, Cc), st.bits)), name
    if debug:
        for L in st.layers:
            if L.kind == "pool":
                continue
            y, yr = N(g.debug["y:" + L.name]), ref["y:" + L.name]
            assert np.array_equal(y, yr), L.name
    return g, ref


def assert_not_degenerate(st, ref):
    # random weights must not drive the stack into a single code
    for name in st.tensor_shapes():
        assert len(np.unique(ref[name])) >= min(4, 2 ** st.bits), name


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("w_offset", [0.0, 0.5])
def test_tiny_stack_every_layer(dsq, bits, w_offset):
    st = dsq_inputs.tiny_stack(bits=bits)
    compare_stack(st, 9, st.batch, w_offset)


def test_tiny_stack_plain_launches(dsq):
    """Same codes with programmatic dependent launch switched off."""
    st = dsq_inputs.tiny_stack(bits=4)
    dsq.dsq_set_dependent_launch(0)
    try:
        compare_stack(st, 9, st.batch, 0.5, debug=False)
    finally:
        dsq.dsq_set_dependent_launch(1)


def test_resnet18_stack_graph_replay_matches_eager(dsq):
    """The captured call sequence (dependent launches become programmatic graph
    edges) reproduces the eager pass bit for bit, replay after replay."""
    from paper_1908_05033_b200.stack import GpuStack
    st = dsq_inputs.resnet18_stack(batch=4)
    x = T(dsq_inputs.stack_input(st, batch=4, workload_id=3))
    params = dsq_inputs.stack_params(st, workload_id=3)
    g = GpuStack(st, params, batch=4)
    eager = g.forward(x).clone()
    names = list(st.tensor_shapes())
    want = {n: g.codes[n].clone() for n in names}
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr, stream=side):
            g.forward(x)
    torch.cuda.synchronize()
    for _ in range(3):
        for n in names:
            g.codes[n].fill_(0xFF)
        gr.replay()
        torch.cuda.synchronize()
        g.check()
        for n in names:
            assert torch.equal(g.codes[n], want[n]), n
    assert torch.equal(g.codes[st.out], eager)


def test_resnet18_stack_batch1_every_layer(dsq):
    st = dsq_inputs.resnet18_stack()
    _, ref = compare_stack(st, 3, 1)
    assert_not_degenerate(st, ref)


def test_resnet18_stack_3bit_batch1_every_layer(dsq):
    """The ResNet-18-shaped stack at 3 bits (the paper's Table 8 times 3-bit
    convolutions on its layer shapes): 3x3 stride-1 layers on the window
    kernel or the im2col kernel, strided and 1x1 layers on the im2col kernel
    with one K step group per filter tap."""
    st = dsq_inputs.resnet18_stack(bits=3)
    _, ref = compare_stack(st, 3, 1)
    assert_not_degenerate(st, ref)


def test_mobilenetv2_stack_batch1_every_layer(dsq):
    st = dsq_inputs.mobilenetv2_stack()
    _, ref = compare_stack(st, 4, 1)
    assert_not_degenerate(st, ref)


def test_vgg16_stack_reduced_every_layer(dsq):
    # 2-bit, 64x64 input (about 1.2 GMAC per image for the oracle)
    st = dsq_inputs.vgg16_stack(hw=64)
    _, ref = compare_stack(st, 5, 1)
    assert_not_degenerate(st, ref)


def test_resnet18_full_batch_sampled_images(dsq):
    """The launch configuration the benchmark times (batch 64): images are
    independent, so the oracle recomputes two of them alone and every layer's
    codes for those images must match."""
    from paper_1908_05033_b200.stack import GpuStack
    st = dsq_inputs.resnet18_stack()
    x = dsq_inputs.stack_input(st, workload_id=3)
    params = dsq_inputs.stack_params(st, workload_id=3)
    g = GpuStack(st, params)
    g.forward(T(x))
    g.check()
    for img in (0, 41):
        ref = ostack.run_stack(st, x[img:img + 1], params,
                               keep=list(st.tensor_shapes()))
        for name in st.tensor_shapes():
            assert np.array_equal(N(g.unpack(name)[img:img + 1]), ref[name]), name
    # a CUDA-graph replay of the same calls gives identical bits
    out1 = g.codes[st.out].clone()
    xs = T(x)
    graph = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        g.forward(xs)
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=s):
            g.forward(xs)
    g.codes[st.out].zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out1, g.codes[st.out])
    g.check()


def _unpack_image(dsq, g, name, img):
    H, W, Cc = g.shapes[name]
    packed = g.codes[name][img:img + 1].reshape(H * W, -1).contiguous()
    return N(dsq.dsq_unpack(packed, H * W, Cc, g.bits, False)).reshape(1, H, W, Cc)


def _full_batch_sampled(dsq, st, wid, images):
    """One forward pass at the batch and image size the benchmark times; the
    oracle recomputes single images alone (images are independent) and every
    code tensor of every layer must match for them."""
    from paper_1908_05033_b200.stack import GpuStack
    x = dsq_inputs.stack_input(st, workload_id=wid)
    params = dsq_inputs.stack_params(st, workload_id=wid)
    g = GpuStack(st, params)
    assert g.batch == st.batch
    g.forward(T(x))
    g.check()
    names = list(st.tensor_shapes())
    for img in images:
        ref = ostack.run_stack(st, x[img:img + 1], params, keep=names)
        for name in names:
            assert np.array_equal(_unpack_image(dsq, g, name, img), ref[name]), (img, name)
    return g


def test_mobilenetv2_full_batch_sampled_images(dsq):
    """MobileNetV2-shaped stack at batch 64 on 112x112x32, as timed."""
    st = dsq_inputs.mobilenetv2_stack()
    assert st.batch == 64 and st.in_shape == (112, 112, 32)
    _full_batch_sampled(dsq, st, 4, (0, 37, 63))


def test_vgg16_full_size_sampled_images(dsq):
    """VGG-16-shaped 2-bit stack at batch 32 on 224x224x64, as timed."""
    st = dsq_inputs.vgg16_stack()
    assert st.batch == 32 and st.in_shape == (224, 224, 64)
    _full_batch_sampled(dsq, st, 5, (0, 21))
