"""The allocation-free partial-gradient entry point against the ordinary one and the CPU oracle.

Collected last on purpose (file name): a run that stops at the first failure has then already run
every other test.  The entry point serves callers that cannot obtain device memory for the
residual workspace -- code inside a latency-critical loop where an allocation would stall the GPU,
a process that has given all device memory to someone else's pool, a plug-in handed only pointers
and a stream -- by keeping that workspace in a fixed array inside the library.
"""
import numpy as np
import pytest

from oracle import cr_oracle as O
from paper_1902_01981_b200 import binding as B
from paper_1902_01981_b200 import build as cr_build
from paper_1902_01981_b200 import inputs
from tests.gpu_common import REL_L2_BAR, rel_l2

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def test_static_scratch_variant_matches_workspace_variant_twice():
    cr_build.build()
    assert torch.cuda.is_available()
    n, L, s, P, d, rows = 4, 2, 1, 24, 1000, 50
    plan = B.cr_plan_create(n, L, s, P, d, code=B.CR_CODE_CYCLIC_RANDOM, device=0)
    try:
        N, m = B.cr_plan_num_nodes(plan), B.cr_plan_load(plan)
        assert N * m * rows <= B.cr_partial_gradients_static_capacity()
        X, y, _ = inputs.linreg_partitions(P, rows, d, seed=31, x_std=1.0 / np.sqrt(d))
        X_dev, y_dev = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda()
        ws = torch.empty(B.cr_partial_gradients_workspace_bytes(plan, rows), dtype=torch.uint8, device="cuda")
        # two calls in a row, on different models: the second finds the first one's residuals in the
        # shared array and must not be affected by them
        for call, seed in enumerate((32, 33)):
            w = inputs.model_vector(d, seed)
            w_dev = torch.from_numpy(w).cuda()
            want = torch.zeros((N, m, d), device="cuda")
            got = torch.full((N, m, d), float("nan"), device="cuda")
            B.cr_partial_gradients(plan, X_dev, y_dev, rows, w_dev, want, ws)
            B.cr_partial_gradients_static(plan, X_dev, y_dev, rows, w_dev, got)
            torch.cuda.synchronize()
            want_h, got_h = want.cpu().numpy(), got.cpu().numpy()
            assert np.isfinite(got_h).all()
            worst = max(rel_l2(got_h[v, j], want_h[v, j]) for v in range(N) for j in range(m))
            assert worst <= REL_L2_BAR, f"call {call}: {worst:.2e}"
            # and against the definition, X_p^T (X_p w - y_p) in fp64, slot by slot
            part = B.slot_partitions(plan)
            truth = [O.partial_gradient_linreg(X[p], y[p], w) for p in range(P)]
            worst = max(rel_l2(got_h[v, j], truth[part[v, j]]) for v in range(N) for j in range(m))
            assert worst <= REL_L2_BAR, f"call {call} against the oracle: {worst:.2e}"
        # a problem beyond the fixed scratch is refused before anything is launched
        too_many = B.cr_partial_gradients_static_capacity() // (N * m) + 1
        launches = B.cr_plan_launch_count(plan)
        with pytest.raises(B.CodedReduceError) as e:
            B.cr_partial_gradients_static(plan, X_dev, y_dev, too_many, w_dev, got)
        assert e.value.status == B.CR_ERR_OOM
        assert B.cr_plan_launch_count(plan) == launches
    finally:
        B.cr_plan_destroy(plan)
