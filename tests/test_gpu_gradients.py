"""Partial and coded gradients for both losses, and the aggregation fed from coded gradients."""
import numpy as np
import pytest

from oracle import cr_oracle as O
from paper_1902_01981_b200 import binding as B
from paper_1902_01981_b200 import build as cr_build
from paper_1902_01981_b200 import inputs
from tests.gpu_common import REL_L2_BAR, check_slot_table, make_plan, rel_l2

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


@pytest.fixture(scope="module", autouse=True)
def built():
    cr_build.build()
    assert torch.cuda.is_available()


def oracle_parts(loss, X, y, w):
    fn = O.partial_gradient_linreg if loss == B.CR_LOSS_SQUARED else O.partial_gradient_logistic
    return np.stack([fn(X[p], y[p], w) for p in range(X.shape[0])])


def make_data(loss, P, rows, d, seed):
    if loss == B.CR_LOSS_SQUARED:
        X, y, _ = inputs.linreg_partitions(P, rows, d, seed, x_std=1.0 / np.sqrt(d))
    else:
        X, y, _ = inputs.logistic_partitions(P, rows, d, seed, x_std=1.0 / np.sqrt(d))
    return X, y, inputs.model_vector(d, seed + 1)


CASES = [dict(n=3, L=2, s=1, P=15, d=512, code="printed_3_1", rows=37),      # one CTA per item, ragged blocks
         dict(n=4, L=2, s=1, P=24, d=1000, code="cyclic", rows=100),          # cluster of CTAs, d not a power of two
         dict(n=4, L=2, s=1, P=48, d=4096, code="cyclic", rows=64),
         dict(n=5, L=1, s=2, P=5, d=8192, code="cyclic", rows=50),            # widest one-pass case
         dict(n=4, L=2, s=1, P=24, d=2048, code="cyclic", rows=33),           # two column groups per thread, six-row blocks, ragged
         dict(n=3, L=2, s=1, P=15, d=6000, code="printed_3_1", rows=25),      # six groups, the last one partly beyond d
         dict(n=4, L=2, s=1, P=24, d=6500, code="cyclic", rows=19),           # seven groups, one-row blocks (a model size of Section V)
         dict(n=3, L=2, s=1, P=15, d=1027, code="printed_3_1", rows=21)]      # two-pass path (d % 4 != 0)


@pytest.mark.parametrize("loss", [B.CR_LOSS_SQUARED, B.CR_LOSS_LOGISTIC])
@pytest.mark.parametrize("cfg", CASES)
def test_partial_and_coded_gradients(cfg, loss):
    n, L, s, P, d, rows = cfg["n"], cfg["L"], cfg["s"], cfg["P"], cfg["d"], cfg["rows"]
    plan = make_plan(cfg)
    try:
        code, local = check_slot_table(plan, cfg)
        X, y, w = make_data(loss, P, rows, d, seed=7)
        parts = oracle_parts(loss, X, y, w)
        N, m = B.cr_plan_num_nodes(plan), B.cr_plan_load(plan)
        X_dev, y_dev, w_dev = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda(), torch.from_numpy(w).cuda()
        G_slots = torch.full((N, m, d), float("nan"), device="cuda")
        ws = torch.empty(B.cr_partial_gradients_workspace_bytes(plan, rows), dtype=torch.uint8, device="cuda")
        B.cr_partial_gradients_loss(plan, loss, X_dev, y_dev, rows, w_dev, G_slots, ws)
        torch.cuda.synchronize()
        got = G_slots.cpu().numpy()
        part = B.slot_partitions(plan)
        for v in range(N):
            for j in range(m):
                assert rel_l2(got[v, j], parts[part[v, j]]) <= REL_L2_BAR
        if d % 4 != 0:
            E = torch.zeros((N, d), device="cuda")
            with pytest.raises(B.CodedReduceError) as e:
                B.cr_coded_gradients(plan, loss, X_dev, y_dev, rows, w_dev, E)
            assert e.value.status == B.CR_ERR_INVALID_ARG
            return
        # coded gradients in one step, against the oracle's encode of the oracle's partition gradients
        E = torch.full((N, d), float("nan"), device="cuda")
        B.cr_coded_gradients(plan, loss, X_dev, y_dev, rows, w_dev, E)
        torch.cuda.synchronize()
        E_or = O.encode_all(local, parts)
        E_host = E.cpu().numpy()
        scale = max(np.linalg.norm(parts[p]) for p in range(P))
        for v in range(N):       # a coded gradient may cancel: measure against the size of its terms
            assert np.linalg.norm(E_host[v] - E_or[v]) <= REL_L2_BAR * max(np.linalg.norm(E_or[v]), scale)
        # aggregation fed from the coded gradients
        masks = inputs.straggler_masks(n, L, s, 6, seed=3)
        out = torch.zeros((6, d), device="cuda")
        for flags in (B.CR_AGG_FUSED, B.CR_AGG_FUSED_LDG):
            out.zero_()
            B.cr_aggregate(plan, E, masks, out, flags | B.CR_AGG_FROM_CODED)
            one = torch.zeros((1, d), device="cuda")
            B.cr_aggregate(plan, E, masks[5], one, flags | B.CR_AGG_FROM_CODED)
            torch.cuda.synchronize()
            for b in range(6):
                assert rel_l2(out[b].cpu().numpy(), O.execute(code, local, parts, masks[b])) <= REL_L2_BAR
            assert rel_l2(one[0].cpu().numpy(), O.full_gradient(parts)) <= REL_L2_BAR
        ws2 = torch.empty(B.cr_aggregate_workspace_bytes(plan, 1, B.CR_AGG_UNFUSED), dtype=torch.uint8, device="cuda")
        with pytest.raises(B.CodedReduceError):
            B.cr_aggregate(plan, E, masks[0], one, B.CR_AGG_UNFUSED | B.CR_AGG_FROM_CODED, ws2)
        assert B.cr_plan_device_status(plan) == B.CR_OK
    finally:
        B.cr_plan_destroy(plan)


def test_logistic_regression_descent_on_paper_shaped_data():
    """(12,2) tree, one straggler per group, 168 partitions of 39 samples, 5004 features: gradient
    descent with coded gradients; every iterate's gradient against the oracle at the same iterate."""
    cfg = inputs.CONFIGS["cfg_logit"]
    n, L, s, P, d, rows = cfg["n"], cfg["L"], cfg["s"], cfg["P"], cfg["d"], cfg["rows"]
    plan = make_plan(cfg)
    try:
        code, local = check_slot_table(plan, cfg)
        X, y, w_star = inputs.logistic_partitions(P, rows, d, cfg["seed"], cfg["x_std"])
        X64, y64 = X.astype(np.float64), y.astype(np.float64)
        N = B.cr_plan_num_nodes(plan)
        X_dev, y_dev = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda()
        w_dev = torch.zeros(d, device="cuda")
        E = torch.zeros((N, d), device="cuda")
        out = torch.zeros((1, d), device="cuda")
        masks = inputs.straggler_masks(n, L, s, cfg["iters"], cfg["mask_seed"])
        losses = []
        for t in range(cfg["iters"]):
            w_t = w_dev.cpu().numpy()
            B.cr_coded_gradients(plan, B.CR_LOSS_LOGISTIC, X_dev, y_dev, rows, w_dev, E)
            B.cr_aggregate(plan, E, masks[t], out, B.CR_AGG_FUSED | B.CR_AGG_FROM_CODED)
            torch.cuda.synchronize()
            if t % 4 == 0 or t == cfg["iters"] - 1:
                parts = np.stack([O.partial_gradient_logistic(X64[p], y64[p], w_t) for p in range(P)])
                assert rel_l2(out[0].cpu().numpy(), O.execute(code, local, parts, masks[t])) <= REL_L2_BAR
                assert rel_l2(out[0].cpu().numpy(), O.full_gradient(parts)) <= REL_L2_BAR
            losses.append(sum(O.loss_logistic(X64[p], y64[p], w_t) for p in range(P)))
            w_dev -= (cfg["lr"] / P) * out[0] * 10.0
        assert np.all(np.diff(losses) < 0)
        assert B.cr_plan_device_status(plan) == B.CR_OK
    finally:
        B.cr_plan_destroy(plan)


def test_a_step_captured_in_a_cuda_graph_equals_the_direct_step():
    """Gradients + scheduled aggregation enqueue kernels only (no copy, no wait, no allocation), so a step
    can be captured in a CUDA graph; its replay must give the bits of the direct calls, and the oracle's
    gradient within the bar."""
    cfg = dict(n=4, L=2, s=1, P=24, d=1000, code="cyclic", rows=100)
    P, d, rows = cfg["P"], cfg["d"], cfg["rows"]
    plan = make_plan(cfg)
    try:
        code, local = check_slot_table(plan, cfg)
        X, y, w = make_data(B.CR_LOSS_SQUARED, P, rows, d, seed=11)
        N, m = B.cr_plan_num_nodes(plan), B.cr_plan_load(plan)
        X_dev, y_dev, w_dev = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda(), torch.from_numpy(w).cuda()
        G_slots = torch.zeros((N, m, d), device="cuda")
        ws = torch.empty(max(16, B.cr_partial_gradients_workspace_bytes(plan, rows)), dtype=torch.uint8, device="cuda")
        mask = inputs.straggler_masks(cfg["n"], cfg["L"], cfg["s"], 1, seed=5, exactly_s=True)[0]
        direct = torch.zeros((1, d), device="cuda")
        B.cr_partial_gradients_loss(plan, B.CR_LOSS_SQUARED, X_dev, y_dev, rows, w_dev, G_slots, ws)
        B.cr_aggregate(plan, G_slots, mask, direct, B.CR_AGG_FUSED)
        torch.cuda.synchronize()
        sched = B.cr_schedule_create(plan, mask, B.CR_AGG_FUSED)
        out = torch.zeros((1, d), device="cuda")
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            cs = torch.cuda.current_stream()
            B.cr_partial_gradients_loss(plan, B.CR_LOSS_SQUARED, X_dev, y_dev, rows, w_dev, G_slots, ws, cs)
            B.cr_aggregate_scheduled(plan, G_slots, sched, out, None, cs)
        G_slots.zero_()
        out.zero_()
        for _ in range(2):
            graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, direct)
        parts = oracle_parts(B.CR_LOSS_SQUARED, X, y, w)
        assert rel_l2(out[0].cpu().numpy(), O.execute(code, local, parts, mask)) <= REL_L2_BAR
        assert B.cr_plan_device_status(plan) == B.CR_OK
        B.cr_schedule_destroy(sched)
    finally:
        B.cr_plan_destroy(plan)
