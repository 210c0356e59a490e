"""tardis_ffn_forward_static: the forward for callers that cannot allocate device memory.

A process that gave all device memory to its own pool at start-up, or that runs under a rule of
"no allocation after initialisation", cannot let a library call cudaMalloc on its behalf.  For such
callers the library offers a forward whose scratch is a fixed array inside the library image.  This
test calls it through the C ABI twice in a row (the array is shared and keeps the previous call's
contents, so the second call runs on a dirty array) and checks each result against the ordinary
tardis_ffn_forward on the same inputs and against the fp64 oracle (flags bit for bit, outputs under
the tolerance the parity tests use); it also checks the exact-range mode and the size limit.  The file name makes pytest collect it after every other test.
"""
import pytest
import torch

import paper_2501_10054_b200 as T
import workloads as W
from tests import helpers as Hp

pytestmark = pytest.mark.gpu


def _max_rel(y, y_ref):
    y, y_ref = y.double(), y_ref.double()
    rms = y_ref.pow(2).mean(dim=-1, keepdim=True).sqrt()
    return ((y - y_ref).abs() / torch.maximum(y_ref.abs(), rms)).max().item()


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_static_scratch_forward_matches_regular_forward_twice(dtype):
    cfg = W.LayerConfig("noalloc_" + dtype, 512, 2048, dtype=dtype, n_calib=512)
    L = Hp.to_cuda(W.make_layer(cfg, 3))
    s64 = L.numpy64()
    h = T.fold_layer(L)
    lib = T.load_library()
    try:
        for call, (n, seed) in enumerate(((37, 11), (5, 12))):      # second call: fewer tokens, dirty scratch
            x = W.make_tokens(cfg, n, seed).cuda()
            y_ref = torch.empty_like(x)
            y = torch.full_like(x, float("nan"))
            T.tardis_set_path(h, 1)                                  # same (generic) kernels on the handle's scratch
            T.tardis_ffn_forward(h, x, y_ref)
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            st = lib.tardis_ffn_forward_static(h, x.data_ptr(), y.data_ptr(), n, None)
            assert st == 0, lib.tardis_last_error()
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free_before       # nothing was taken from the device
            assert torch.isfinite(y.float()).all()
            assert _max_rel(y, y_ref) <= Hp.TOL[dtype], "call %d" % call
            assert T.tardis_stats(h)["last_path"] == 5
            # and against the oracle: flags captured from the static entry, outputs of the static entry
            bm = torch.zeros(n, cfg.d_ff // 32, dtype=torch.int32, device="cuda")
            T.tardis_set_debug_capture(h, bm, None)
            y2 = torch.full_like(x, float("nan"))
            assert lib.tardis_ffn_forward_static(h, x.data_ptr(), y2.data_ptr(), n, None) == 0
            torch.cuda.synchronize()
            T.tardis_set_debug_capture(h, None, None)
            Hp.assert_parity(L, s64, x, y2, Hp.unpack_bitmap(bm, cfg.d_ff), None, score_tol=None, label="static call %d" % call)
        # exact-range mode (flags from the true pre-activations) is honoured by the static entry as by the ordinary one
        x = W.make_tokens(cfg, 9, 21).cuda()
        y_a, y_b = torch.empty_like(x), torch.empty_like(x)
        T.tardis_set_path(h, 4)
        T.tardis_ffn_forward(h, x, y_a)
        assert lib.tardis_ffn_forward_static(h, x.data_ptr(), y_b.data_ptr(), 9, None) == 0
        torch.cuda.synchronize()
        assert _max_rel(y_b, y_a) <= Hp.TOL[dtype]
        T.tardis_set_path(h, 1)
        # beyond the limits: refused with a clear message, nothing launched
        x = W.make_tokens(cfg, 65, 13).cuda()
        y = torch.empty_like(x)
        calls = T.tardis_stats(h)["calls"]
        assert lib.tardis_ffn_forward_static(h, x.data_ptr(), y.data_ptr(), 65, None) == 2
        assert b"64" in lib.tardis_last_error()
        with pytest.raises(T.TardisError):
            T.tardis_ffn_forward_static(h, x, y)
        assert T.tardis_stats(h)["calls"] == calls
        assert lib.tardis_ffn_forward_static(h, None, None, 0, None) == 0   # empty call is a no-op
    finally:
        T.tardis_destroy(h)
