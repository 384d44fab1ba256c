"""The time-out path of the attention kernel, exercised without hanging or faulting anything.

Every device-side wait of the kernel is bounded: when one runs out, the thread block records
(code, block, site, iteration) in the workspace's status block, raises a block-wide abort flag,
lets its roles leave in order (copies in flight land, issued tensor-core work completes, tensor
memory is freed) and the blocks that start later leave at once; `avggt_check_status` then returns
AVGGT_ERR_DEVICE_TIMEOUT.  A second build of the same sources (`libavggt_waittest.so`: a 0.5 ms
limit, and the first thread block's producer leaves out one K tile, i.e. a flag that nothing
sets) makes such a wait run out.  The product library does not contain that switch.
"""

import ctypes

import numpy as np
import pytest
import torch

import paper_2512_02541_b200 as P
from oracle import avggt_oracle as orc
from paper_2512_02541_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu


def _forward(L, params, Q, K, V, layer, O):
    """build_kv + global_attn through the library handle L, on the layer's buffers."""
    vp = ctypes.c_void_p
    st = vp(torch.cuda.current_stream().cuda_stream)
    p = ctypes.byref(params)
    rc = L.avggt_build_kv(p, vp(K.data_ptr()), vp(V.data_ptr()), vp(layer.Kc.data_ptr()), vp(layer.Vc.data_ptr()),
                          vp(layer.idx.data_ptr()), vp(layer.kmean.data_ptr()), vp(layer.vmean.data_ptr()),
                          vp(layer.build_ws.data_ptr()), layer.build_ws.numel(), st)
    assert rc == 0
    rc = L.avggt_global_attn(p, vp(Q.data_ptr()), vp(K.data_ptr()), vp(V.data_ptr()), vp(layer.Kc.data_ptr()),
                             vp(layer.Vc.data_ptr()), vp(layer.kmean.data_ptr()), vp(layer.vmean.data_ptr()),
                             vp(O.data_ptr()), None, vp(layer.attn_ws.data_ptr()), layer.attn_ws.numel(), st)
    assert rc == 0
    torch.cuda.synchronize()
    detail = (ctypes.c_uint32 * 4)()
    return L.avggt_check_status(vp(layer.attn_ws.data_ptr()), detail), tuple(detail)


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    # 100 frames of 261 tokens, 16 heads: 1632 thread blocks of 104 key tiles each, about eleven waves of ~0.15 ms,
    # so that the first block's wait (0.5 ms) runs out while most blocks have not started yet
    wl = inputs.Workload("wait_limit", 100, 16, 16, 5, 16, 64, 2, 1, 2, "iid")
    params = P.make_params(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma,
                           diag=wl.diag, mean_fill=wl.mean_fill)
    Q, K, V = inputs.make_qkv(wl, seed=0, device="cuda")
    layer = P.SubsampledGlobalAttention(params)
    O = torch.full_like(Q, float("nan"))

    broken = binding.load_library(build.build_wait_test())
    code, detail = _forward(broken, params, Q, K, V, layer, O)
    assert code == binding.AVGGT_ERR_DEVICE_TIMEOUT
    flag, block, site, iteration = detail
    assert flag == 1 and block == 0                       # the first thread block gave up ...
    # ... in whichever of its roles had waited longest on the consequences of the missing K tile: the producer
    # on a ring stage that is never released (sites 10, 11), an MMA issuer on the tile itself (24, 25) or a
    # softmax warp on the scores of step 1 (40, 41); all within the first cycle of the four-stage ring
    assert site in (10, 11, 24, 25, 40, 41) and iteration <= 5
    # the blocks of the last head start after the time-out and leave at once: their rows were never written
    assert torch.isnan(O[:, wl.n_heads - 1].float()).any()

    # the same workspace and buffers through the product library right afterwards: correct output
    good = binding.lib()
    O.fill_(float("nan"))
    code, detail = _forward(good, params, Q, K, V, layer, O)
    assert code == 0 and detail[0] == 0
    assert torch.isfinite(O.float()).all()
    ocfg = orc.SGAConfig(wl.n_frames, wl.grid_h, wl.grid_w, wl.n_special, wl.n_heads, wl.head_dim, wl.sigma,
                         diag=bool(wl.diag), mean_fill=wl.mean_fill)
    Qh, Kh, Vh = (t.float().cpu().numpy() for t in (Q, K, V))
    rows = inputs.sample_rows(wl, 256).numpy()
    want = orc.global_attn_blocked(ocfg, Qh, Kh, Vh, rows)
    err = np.abs(O[torch.as_tensor(rows, device="cuda")].float().cpu().numpy().astype(np.float64) - want)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3
