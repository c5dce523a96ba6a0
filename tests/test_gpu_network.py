"""Whole-network replay: the YOLOv5s-shaped backbone + neck chained on the GPU (57 pattern convolutions and the
glue kernels, all through the C ABI) against the same program in the CPU oracle on a small input.  Every layer
rounds to bf16, and a one-ulp difference early on changes later roundings, so the chained error is reported and
held to a looser bound than the per-layer tests."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from oracle import rtoss_oracle as orc
    from paper_2303_02191_b200 import synth
    from paper_2303_02191_b200.yolov5s_net import GpuNet
    import gpu_util as gu
    import net_oracle


def test_chained_yolov5s_shaped_network_small_input():
    N, H0 = 2, 96
    x = synth.activations(70, 1, N, 3, H0, H0)
    net = GpuNet(gu.ctx(), N, H0, H0, k=4, seed=3)
    net.set_input(synth.round_like(x, "bf16"))
    net.run()                  # the first pass goes call by call (it finds out which fused calls the library takes)
    torch.cuda.synchronize()
    one_by_one = net.outputs()
    net.run()                  # from then on independent convolutions share launches
    torch.cuda.synchronize()
    assert gu.ctx().rtoss_device_status() == 0
    assert max(len(r) for r in net.rounds) >= 2
    got = net.outputs()
    ref = net_oracle.oracle_forward(x, H0, H0, k=4, seed=3)
    for name in ("o3", "o4", "o5"):   # a shared launch never cuts a layer along K, a single one may: other fp32 summation order
        assert orc.rel_err(got[name], one_by_one[name]) <= 0.05
    for name in ("o3", "o4", "o5"):
        err = orc.rel_err(got[name], ref[name])
        print(name, got[name].shape, "chained relative error %.4f" % err)
        assert got[name].shape == ref[name].shape
        assert err <= 0.1
        assert np.mean(np.abs(got[name] - ref[name])) <= 0.01 * np.sqrt(np.mean(ref[name] ** 2)) + 1e-6
    # dependent convolutions sharing launches (rtoss_conv_chain): far fewer launches, the same network
    net.t["o3"].fill_(float("nan"))
    net.run(chained=True)
    torch.cuda.synchronize()
    assert gu.ctx().rtoss_device_status() == 0
    chained = net.outputs()
    for name in ("o3", "o4", "o5"):
        assert orc.rel_err(chained[name], one_by_one[name]) <= 0.05
        assert orc.rel_err(chained[name], ref[name]) <= 0.1
    # replay through a CUDA graph gives the same bits as the eager run
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        net.run()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    with torch.cuda.graph(g):
        net.run()
    g.replay()
    torch.cuda.synchronize()
    again = net.outputs()
    for name in ("o3", "o4", "o5"):
        assert np.array_equal(again[name], got[name])
    # the runs above add the seven bottleneck shortcuts inside the convolutions; separate adds give the same bits
    assert sum(op[0] == "convres" for op in net.ops) == 7 and len(net.unfused) == 0
    plain = GpuNet(gu.ctx(), N, H0, H0, k=4, seed=3, fuse_residual=False)
    plain.set_input(synth.round_like(x, "bf16"))
    plain.run(grouped=False)
    torch.cuda.synchronize()
    sep = plain.outputs()
    for name in ("o3", "o4", "o5"):
        assert np.array_equal(sep[name], one_by_one[name]), name
    plain.close()
    net.close()


def test_chained_retinanet_shaped_network_small_input():
    """The RetinaNet ResNet-50-FPN-shaped program (100 convolution calls on 68 weight tensors, residual adds,
    top-down pyramid, towers with weights shared across the levels) against the same program in the CPU oracle."""
    from paper_2303_02191_b200 import retinanet_net
    N, H0, W0 = 1, 64, 96
    x = synth.activations(71, 1, N, 64, H0 // 4, W0 // 4)
    net = retinanet_net.GpuNet(gu.ctx(), N, H0, W0, k=4, seed=5)
    net.set_input(synth.round_like(x, "bf16"))
    net.run()                  # call by call
    torch.cuda.synchronize()
    one_by_one = net.outputs()
    net.run()                  # independent convolutions (tower layers over the levels, both towers, ...) share launches
    torch.cuda.synchronize()
    assert gu.ctx().rtoss_device_status() == 0
    assert max(len(r) for r in net.rounds) >= 6
    got = net.outputs()
    for name in net.output_names:
        assert orc.rel_err(got[name], one_by_one[name]) <= 0.05
    ref = net_oracle.oracle_forward_retinanet(x, H0, W0, k=4, seed=5)
    assert len(got) == 10
    for name in net.output_names:
        err = orc.rel_err(got[name], ref[name])
        print(name, got[name].shape, "chained relative error %.4f" % err)
        assert got[name].shape == ref[name].shape
        assert err <= 0.1
        assert np.mean(np.abs(got[name] - ref[name])) <= 0.01 * np.sqrt(np.mean(ref[name] ** 2)) + 1e-6
    # whole stages of bottleneck blocks and successive tower layers in single launches
    for name in net.output_names:
        net.t[name].fill_(float("nan"))
    net.run(chained=True)
    torch.cuda.synchronize()
    assert gu.ctx().rtoss_device_status() == 0
    # (no claim on the number of launches: at this input size the library keeps most layers alone, cut along K)
    chained = net.outputs()
    for name in net.output_names:   # (fifty bf16 layers deep, other tile plans: held to the bound against the oracle)
        assert orc.rel_err(chained[name], one_by_one[name]) <= 0.1
        assert orc.rel_err(chained[name], ref[name]) <= 0.1
    net.run(chained=True)
    torch.cuda.synchronize()
    again = net.outputs()
    for name in net.output_names:
        assert np.array_equal(again[name], chained[name])
    # the run above adds the residuals inside the convolutions; separate add kernels give the same bits
    assert sum(op[0] == "convres" for op in net.ops) == 18 and len(net.unfused) == 0
    plain = retinanet_net.GpuNet(gu.ctx(), N, H0, W0, k=4, seed=5, fuse_residual=False)
    plain.set_input(synth.round_like(x, "bf16"))
    plain.run(grouped=False)
    torch.cuda.synchronize()
    sep = plain.outputs()
    for name in net.output_names:
        assert np.array_equal(sep[name], one_by_one[name]), name
    plain.close()
    net.close()
