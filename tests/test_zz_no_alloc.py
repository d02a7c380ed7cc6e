"""nb_step_static, the entry point for callers that cannot allocate device memory, checked through
the C ABI against the ordinary accumulate + step entry points, and against the CPU oracle, on two
iterations in a row; the second call must leave the amount of free device memory unchanged.

Collected last (file name) so that a run that stops at the first failure has already run every
other test.  It relies on nothing another test leaves behind: the library's fixed accumulator is
fully overwritten by each call before it is read."""
import numpy as np
import pytest

from oracle import nb_oracle as O
from paper_2211_00889_b200 import workloads as WL
from tests import _harness as H

pytestmark = pytest.mark.gpu


def test_static_entry_point_matches_context_path_on_two_calls_in_a_row():
    import torch
    from paper_2211_00889_b200.build import build_library
    build_library()
    from paper_2211_00889_b200 import binding as B

    for name, P in (("cfg2_allreduce_resnet18", 3 * 1024 + 7), ("cfg5_scale_allreduce", 2 * 1024 + 40)):
        w = WL.scaled(WL.WORKLOADS[name], P, steps=2)
        ld = (P + 3) // 4 * 4
        assert w.K * ld <= B.NB_STATIC_MAX_ELEMS
        x0 = WL.init_params(w)
        ctx = B.context_for(w)                                  # the existing entry points
        ctx.set_params(torch.from_numpy(x0).cuda())
        orc = O.Oracle(w.K, P, w.M, w.lr, w.mom, "allreduce")   # independent of both entry points
        orc.set_params(x0)
        X = torch.zeros((w.K, ld), dtype=torch.float32, device="cuda")   # the caller's own memory
        X[:, :P] = torch.from_numpy(x0).cuda()
        V = torch.zeros_like(X)
        for t in range(2):                                      # two calls in a row share the array
            n = H.lib_counts(B, w, t)
            payload, values = WL.gradients_np(w, t)
            g = H.to_device(payload)
            ctx.accumulate(g, n)
            ctx.step()
            orc.step(values, n.tolist())
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            B.step_static(X, V, g, n, P, w.M, w.lr, w.mom)
            torch.cuda.synchronize()
            if t > 0:      # the first call on a device may load the library's code and the fixed array
                assert torch.cuda.mem_get_info()[0] == free_before, "nb_step_static changed the free device memory"
            H.assert_close(X[:, :P].cpu().numpy(), orc.X, H.TOL_SAME_INPUT, "X vs oracle, call %d" % t)
            H.assert_close(V[:, :P].cpu().numpy(), orc.V, H.TOL_SAME_INPUT, "V vs oracle, call %d" % t)
            want_x, want_v = ctx.get_params(device="cuda"), ctx.get_momentum(device="cuda")
            H.assert_close(X[:, :P].cpu().numpy(), want_x.cpu().numpy(), H.TOL_SAME_INPUT, "X call %d" % t)
            H.assert_close(V[:, :P].cpu().numpy(), want_v.cpu().numpy(), H.TOL_SAME_INPUT, "V call %d" % t)
            assert torch.equal(X[:, :P], want_x) and torch.equal(V[:, :P], want_v)   # same operation sequence
        ctx.close()


def test_static_entry_point_rejects_sizes_beyond_its_fixed_array():
    import torch
    from paper_2211_00889_b200.build import build_library
    build_library()
    from paper_2211_00889_b200 import binding as B

    K, M = 8, 2
    ld = B.NB_STATIC_MAX_ELEMS // K + 4                          # one vector too many
    X = torch.zeros((K, ld), dtype=torch.float32, device="cuda")
    V = torch.zeros_like(X)
    g = torch.zeros((K, M, 16), dtype=torch.float32, device="cuda")
    with pytest.raises(B.NbError) as e:
        B.step_static(X, V, g, [1] * K, 16, M, 0.1, 0.9)
    assert e.value.code == B.NB_ERR_UNSUPPORTED and "NB_STATIC_MAX_ELEMS" in str(e.value)
    with pytest.raises(B.NbError) as e:                          # pitch not a multiple of 4
        B.step_static(X[:, :18].contiguous(), V[:, :18].contiguous(), g, [1] * K, 16, M, 0.1, 0.9)
    assert e.value.code == B.NB_ERR_ARG
    assert float(X.abs().max()) == 0.0                           # nothing was launched
