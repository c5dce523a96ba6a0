"""Tensor path on layers with few tiles and many channel blocks: the channel blocks of a tile are shared out to
the CTAs of a thread-block cluster (split K); every CTA leaves its partial sums in the shared memory of the chunk's
owner (distributed shared memory, between two cluster barriers) and finishes the chunks it owns.  Parity against the
CPU oracle, twice in a row on the same context (nothing of the first call may linger), with every activation, a
channel slice of a wider output, a ragged filter count and both kernel sizes."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from oracle import rtoss_oracle as orc
    from paper_2303_02191_b200 import binding as rt
    from paper_2303_02191_b200 import synth
    import gpu_util as G

CASES = [
    # ksize, Cin, Cout, N, H, W, stride, act, (y_off, y_stride)
    (3, 256, 256, 2, 13, 17, 1, "relu", (0, 0)),
    (3, 256, 256, 1, 7, 9, 1, "none", (0, 0)),
    (3, 512, 128, 1, 20, 20, 1, "silu", (0, 0)),
    (3, 320, 100, 1, 9, 11, 1, "silu", (0, 0)),       # ragged filter count: element stores; five channel blocks in four shares
    (3, 256, 128, 1, 12, 12, 2, "silu", (64, 256)),   # stride 2, channel slice of a wider tensor
    (1, 2048, 512, 1, 7, 9, 1, "relu", (0, 0)),
    (1, 2048, 128, 2, 10, 10, 1, "silu", (0, 0)),
    (3, 256, 256, 4, 25, 34, 1, "relu", (0, 0)),      # sixteen tiles x four shares: 64 CTAs
]


def test_split_k_fp16_and_graph_replay():
    """fp16 data, and the cluster launch captured into a CUDA graph: the replay gives the bits of the eager run."""
    masks = orc.pattern_preset(3, orc.PRESET_CONN4)
    w = synth.kaiming_weights(4, 12, 256, 256, 3)
    b = synth.bias(4, 12, 256)
    x = synth.round_like(synth.activations(4, 12, 2, 256, 13, 17), "f16")
    pid, packed = G.select_pack(w, 3, masks, 3, "f16")
    _, wd, _ = G.oracle_weights(w, 3, masks, 3, "f16")
    ref = orc.conv3x3(x, wd, b, 1, orc.ACT_SILU, orc.DT_F16)
    c = G.ctx()
    xd = G.to_dev(x, "f16", "nhwc")
    bd = torch.from_numpy(b).cuda()
    y = torch.zeros((2, 13, 17, 256), dtype=torch.float16, device="cuda")

    def run():
        c.rtoss_conv3x3_pattern(packed, xd, y, 2, 13, 17, 1, rt.NHWC, rt.ACT_SILU, bd, path=rt.PATH_TENSOR)

    run()
    torch.cuda.synchronize()
    eager = y.clone()
    assert orc.rel_err(G.from_dev(eager, "nhwc"), ref) <= G.TOL["f16"]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        run()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        run()
    y.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(y, eager)
    assert c.rtoss_device_status() == 0
    packed.close()


@pytest.mark.parametrize("ksize,cin,cout,N,H,W,stride,act,ysl", CASES)
def test_split_k_parity(ksize, cin, cout, N, H, W, stride, act, ysl):
    masks = orc.pattern_preset(4, orc.PRESET_CENTRE8)
    w = synth.kaiming_weights(3, 11, cout, cin, ksize)
    b = synth.bias(3, 11, cout)
    x = synth.round_like(synth.activations(3, 11, N, cin, H, W), "bf16")
    pid, packed = G.select_pack(w, ksize, masks, 4, "bf16")
    pid_o, wd, _ = G.oracle_weights(w, ksize, masks, 4, "bf16")
    assert np.array_equal(pid, pid_o.ravel())
    conv = orc.conv3x3 if ksize == 3 else orc.conv1x1
    ref = conv(x, wd, b, stride, {"none": orc.ACT_NONE, "relu": orc.ACT_RELU, "silu": orc.ACT_SILU}[act], orc.DT_BF16)
    for _ in range(2):
        y = G.run_conv(packed, ksize, x, "bf16", stride, act, b, layout="nhwc", y_off=ysl[0], y_stride=ysl[1], path=rt.PATH_TENSOR)
        if ysl[1]:
            y = y[:, ysl[0]:ysl[0] + cout]
        err = orc.rel_err(y, ref)
        assert err <= G.TOL["bf16"], "relative error %g" % err
    assert G.ctx().rtoss_device_status() == 0
    packed.close()
