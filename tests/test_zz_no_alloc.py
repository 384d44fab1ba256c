"""avggt_build_kv_noalloc against avggt_build_kv, through the C ABI.

The no-allocation entry point serves callers that have no device memory to lend as workspace and
may not create any (all of the GPU's memory already belongs to the host program's memory manager,
or cudaMalloc's device-wide synchronisation is not acceptable where the call is made).  Its scratch
is one fixed array inside the library that every call reuses, so the check runs two calls in a row
with different inputs: the second must not be disturbed by what the first left behind.

This file is collected last on purpose (a run that stops at the first failure has then already run
every other test) and must pass alone in a fresh process as well as after the other tests.
"""

import numpy as np
import pytest
import torch

import paper_2512_02541_b200 as P
from oracle import avggt_oracle as orc
from paper_2512_02541_b200 import inputs

pytestmark = pytest.mark.gpu


def _buffers(layer):
    return (torch.full_like(layer.Kc, float("nan")), torch.full_like(layer.Vc, float("nan")),
            torch.full_like(layer.idx, -1), torch.full_like(layer.kmean, float("nan")),
            torch.full_like(layer.vmean, float("nan")))


@pytest.mark.parametrize("wl", [
    inputs.WORKLOADS["tiny_n4_g16_s2"],
    inputs.Workload("noalloc_ragged", 9, 37, 37, 5, 16, 64, 6, 1, 2, "iid"),
])
def test_noalloc_matches_build_kv_twice_in_a_row(wl):
    params = P.make_params(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma,
                           diag=wl.diag, mean_fill=wl.mean_fill)
    layer = P.SubsampledGlobalAttention(params)
    stream = torch.cuda.current_stream().cuda_stream
    for call, seed in enumerate((3, 4)):          # two calls in a row, different data
        _, K, V = inputs.make_qkv(wl, seed=seed, device="cuda")
        if call == 1:
            K = K * 2 + 1                          # shifts the means well away from the first call's
            V = V - 3
        layer.build_kv(K, V)                       # the existing entry point, with a caller workspace
        Kc, Vc, idx, kmean, vmean = _buffers(layer)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        P.avggt_build_kv_noalloc(params, K, V, Kc, Vc, idx, kmean, vmean, stream)
        torch.cuda.synchronize()
        # the call takes no device memory (checked from the second call on: the first one on a device may make
        # the CUDA runtime load the kernels' code)
        if call == 1:
            assert torch.cuda.mem_get_info()[0] == free_before
        assert torch.equal(idx, layer.idx)
        assert torch.equal(Kc.view(torch.int16), layer.Kc.view(torch.int16))      # bit copies
        assert torch.equal(Vc.view(torch.int16), layer.Vc.view(torch.int16))
        # the mean pair is summed over differently sized groups: same tolerance as the parity tests
        for got, want, src in ((kmean, layer.kmean, K), (vmean, layer.vmean, V)):
            scale = max(float(src.float().abs().mean()), 1e-6)
            assert torch.isfinite(got).all()
            assert float((got - want).abs().max()) <= 1e-5 * scale
        # and against the fp64 oracle directly
        ocfg = orc.SGAConfig(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma,
                             diag=bool(wl.diag), mean_fill=wl.mean_fill)
        Kh, Vh = K.float().cpu().numpy(), V.float().cpu().numpy()
        Kc_w, Vc_w, idx_w, kmean_w, vmean_w = orc.build_kv(ocfg, Kh, Vh)
        np.testing.assert_array_equal(idx.cpu().numpy(), idx_w)
        np.testing.assert_array_equal(Kc.float().cpu().numpy().transpose(1, 0, 2).astype(np.float64), Kc_w)
        np.testing.assert_array_equal(Vc.float().cpu().numpy().transpose(1, 0, 2).astype(np.float64), Vc_w)
        for got, want, src in ((kmean, kmean_w, Kh), (vmean, vmean_w, Vh)):
            assert np.abs(got.cpu().numpy().astype(np.float64) - want).max() <= 1e-5 * max(float(np.abs(src).mean()), 1e-6)


def test_noalloc_rejects_problems_beyond_its_fixed_scratch():
    wl = inputs.Workload("too_wide", 2, 6, 6, 5, 32, 64, 4, 1, 2, "iid")      # H * d = 2048 > 1024
    params = P.make_params(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma)
    layer = P.SubsampledGlobalAttention(params)
    _, K, V = inputs.make_qkv(wl, seed=0, device="cuda")
    with pytest.raises(P.AvggtError) as ei:
        P.avggt_build_kv_noalloc(params, K, V, layer.Kc, layer.Vc, layer.idx, layer.kmean, layer.vmean,
                                 torch.cuda.current_stream().cuda_stream)
    assert ei.value.code == -7
    assert "fixed scratch" in str(ei.value)
    torch.cuda.synchronize()
