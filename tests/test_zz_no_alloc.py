"""The allocation-free pruning entry point, rtoss_prune_dense_static.

It serves callers that cannot call cudaMalloc (all device memory already given to their own arena, or
no tolerance for cudaMalloc's device-wide synchronisation): the pattern ids live in a fixed array inside
the library.  Checked here through the C ABI against the allocating chain select -> pack -> to_dense
and against the CPU oracle's W (.) mask, bit for bit, on consecutive calls (a call must not see anything of
the one before in the shared array), for both kernel sizes, also in place (output = input); the size limit
and overlapping arrays must be refused.  Collected last on purpose."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from oracle import rtoss_oracle as orc
    from paper_2303_02191_b200 import binding as rt
    from paper_2303_02191_b200 import synth


def _oracle_pruned(w, ksize, masks):
    """W (.) mask from the CPU oracle; w's values are exact in fp32 whatever its storage type."""
    wf = w.float().cpu().numpy()
    if ksize == 3:
        return orc.mask_3x3(wf, masks, orc.select_3x3(wf, masks))
    w2 = wf.reshape(wf.shape[0], wf.shape[1])
    return orc.mask_1x1(w2, masks, orc.select_1x1(w2, masks)).reshape(wf.shape)


def _chain(ctx, w, ksize, masks, k):
    pid = ctx.rtoss_select_patterns(w, ksize, masks, k)
    packed = ctx.rtoss_pack(w, ksize, masks, k, pid, rt._torch_dtype_code(w))
    dense = packed.to_dense().clone()
    torch.cuda.synchronize()
    packed.close()
    return dense.reshape(w.shape)


def test_static_pruning_matches_the_allocating_chain_twice_in_a_row():
    ctx = rt.Context(0)
    masks3 = rt.rtoss_pattern_preset(3, rt.PRESET_CONN4)
    masks4 = rt.rtoss_pattern_preset(4, rt.PRESET_CENTRE8)
    calls = [
        (torch.from_numpy(synth.kaiming_weights(31, 1, 96, 80, 3)).cuda(), 3, masks3, 3),                          # 7680 kernels, fp32
        (torch.from_numpy(synth.kaiming_weights(31, 2, 40, 56, 3)).cuda(), 3, masks4, 4),                          # fewer kernels than the call before
        (torch.from_numpy(synth.kaiming_weights(31, 3, 128, 256, 1)).cuda().to(torch.bfloat16), 1, masks3, 3),     # 1x1, bf16, 8 left-over weights
        (torch.from_numpy(synth.kaiming_weights(31, 4, 2, 4, 1)).cuda(), 1, masks3, 3),                            # fewer than nine weights: all pruned
    ]
    for w, ksize, masks, k in calls:
        out = torch.full_like(w, 7.0)
        st, out = rt.rtoss_prune_dense_static(w, ksize, masks, k, out)
        assert st == rt.OK
        torch.cuda.synchronize()
        want = _chain(ctx, w, ksize, masks, k)
        a = out.float().cpu().numpy().view(np.uint32)
        b = want.float().cpu().numpy().view(np.uint32)
        assert np.array_equal(a, b)
        assert np.array_equal(a, _oracle_pruned(w, ksize, masks).view(np.uint32))
        # in place: the output array is the input array
        w2 = w.clone()
        st, same = rt.rtoss_prune_dense_static(w2, ksize, masks, k, w2)
        assert st == rt.OK
        torch.cuda.synchronize()
        assert np.array_equal(w2.float().cpu().numpy().view(np.uint32), b)
        kept = np.count_nonzero(out.float().cpu().numpy().reshape(-1))
        n_k = w.shape[0] * w.shape[1] if ksize == 3 else (w.shape[0] * w.shape[1]) // 9
        assert kept == n_k * k
    ctx.close()


def test_static_pruning_refuses_layers_beyond_its_fixed_array():
    masks = rt.rtoss_pattern_preset(2, rt.PRESET_CONN4)
    w = torch.zeros(1024, 1025, 3, 3, device="cuda", dtype=torch.float16)       # 1 049 600 kernels > 2^20
    st, _ = rt.rtoss_prune_dense_static(w, 3, masks, 2, torch.empty_like(w))
    assert st == 3
    ok = torch.zeros(1024, 1024, 3, 3, device="cuda", dtype=torch.float16)      # exactly 2^20 kernels: accepted
    st, out = rt.rtoss_prune_dense_static(ok, 3, masks, 2, torch.full_like(ok, 1.0))
    torch.cuda.synchronize()
    assert st == rt.OK and not out.any()
    st, _ = rt.rtoss_prune_dense_static(ok, 3, [3, 3], 2, torch.empty_like(ok))  # duplicate mask
    assert st == 2
    # two different arrays that overlap: refused before anything is launched
    flat = torch.zeros(2 * 16 * 16 * 9 + 64, device="cuda")
    a = flat[:16 * 16 * 9].view(16, 16, 3, 3)
    b = flat[64:64 + 16 * 16 * 9].view(16, 16, 3, 3)
    st, _ = rt.rtoss_prune_dense_static(a, 3, masks, 2, b)
    assert st == 1
