"""Partial gradients of K models at once (tensor-core path) against the per-model oracle gradients."""
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


def make_data(loss, P, rows, d, seed):
    """Features rounded to TF32-representable values BEFORE the labels are formed, so that the oracle
    and the tensor cores see the same numbers."""
    x_std = 1.0 / np.sqrt(d)
    if loss == B.CR_LOSS_SQUARED:
        X, _, w_star = inputs.linreg_partitions(P, rows, d, seed, x_std=x_std)
        X = inputs.tf32_representable(X)
        noise = inputs.partition_gradients(P, rows, seed + 100, 0.01)
        y = np.stack([(X[p].astype(np.float64) @ w_star.astype(np.float64) + noise[p]).astype(np.float32)
                      for p in range(P)])
    else:
        X, y, _ = inputs.logistic_partitions(P, rows, d, seed, x_std=x_std)
        X = inputs.tf32_representable(X)
    return X, y


def oracle_parts(loss, X, y, w):
    fn = O.partial_gradient_linreg if loss == B.CR_LOSS_SQUARED else O.partial_gradient_logistic
    return np.stack([fn(X[p], y[p], w) for p in range(X.shape[0])])


CASES = [dict(n=3, L=1, s=1, P=6, d=256, code="printed_3_1", rows=64, K=3),      # one row tile, two column tiles
         dict(n=3, L=1, s=1, P=6, d=1000, code="printed_3_1", rows=200, K=32),   # ragged rows and columns, all models
         dict(n=3, L=2, s=1, P=15, d=36, code="printed_3_1", rows=9, K=1),       # smallest shapes
         dict(n=4, L=2, s=1, P=24, d=5004, code="cyclic", rows=39, K=8),         # shape of the logistic run
         dict(n=4, L=2, s=1, P=48, d=4096, code="cyclic", rows=512, K=16),
         dict(n=3, L=1, s=1, P=6, d=16384, code="printed_3_1", rows=24, K=2),     # long contraction over d
         # partitions of few rows: several items share a 128-row tile (five of 24 rows here, 48 items: a ragged
         # last group), one CTA walks the column tiles of an item
         dict(n=3, L=2, s=1, P=15, d=300, code="printed_3_1", rows=20, K=5),
         dict(n=3, L=1, s=1, P=6, d=520, code="printed_3_1", rows=60, K=4),       # eight k-steps: the head accumulators wrap
         dict(n=12, L=2, s=1, P=168, d=1028, code="cyclic", rows=39, K=32),       # 624 items of 39 rows, three per tile
         dict(n=3, L=1, s=1, P=6, d=132, code="printed_3_1", rows=65, K=2)]       # just above: the general kernels


@pytest.mark.parametrize("loss", [B.CR_LOSS_SQUARED, B.CR_LOSS_LOGISTIC])
@pytest.mark.parametrize("cfg", CASES)
def test_multi_model_gradients(cfg, loss):
    P, d, rows, K = cfg["P"], cfg["d"], cfg["rows"], cfg["K"]
    plan = make_plan(cfg)
    try:
        check_slot_table(plan, cfg)
        X, y = make_data(loss, P, rows, d, seed=11)
        W = inputs.model_matrix(K, d, seed=12)
        N, m = B.cr_plan_num_nodes(plan), B.cr_plan_load(plan)
        part = B.slot_partitions(plan)
        X_dev, y_dev, W_dev = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda(), torch.from_numpy(W).cuda()
        G = torch.full((K, N, m, d), float("nan"), device="cuda")
        R = torch.full((N, m, rows, K), float("nan"), device="cuda")
        ws = torch.empty(B.cr_partial_gradients_multi_workspace_bytes(plan, rows), dtype=torch.uint8, device="cuda")
        B.cr_partial_gradients_multi(plan, loss, X_dev, y_dev, rows, W_dev, K, G, ws, R_out=R)
        torch.cuda.synchronize()
        B.cr_plan_device_status(plan)
        got_R, got_G = R.cpu().numpy(), G.cpu().numpy()
        for k in range(K):
            # residuals first (they locate a mistake: first or second contraction)
            wk = W[k].astype(np.float64)
            for p in sorted(set(part.reshape(-1).tolist())):
                z = X[p].astype(np.float64) @ wk
                want = (z if loss == B.CR_LOSS_SQUARED else 1.0 / (1.0 + np.exp(-z))) - y[p]
                v, j = np.argwhere(part == p)[0]
                assert rel_l2(got_R[v, j, :, k], want) <= REL_L2_BAR, ("residual", k, p)
            parts = oracle_parts(loss, X, y, W[k])
            for v in range(N):
                for j in range(m):
                    assert rel_l2(got_G[k, v, j], parts[part[v, j]]) <= REL_L2_BAR, ("gradient", k, v, j)
    finally:
        B.cr_plan_destroy(plan)


def test_multi_model_gradients_feed_the_aggregation():
    """Each G_multi[k] is a slot buffer: aggregating it gives the full gradient at W[k]."""
    cfg = dict(n=3, L=2, s=1, P=15, d=512, code="printed_3_1", rows=48, K=4)
    P, d, rows, K = cfg["P"], cfg["d"], cfg["rows"], cfg["K"]
    plan = make_plan(cfg)
    try:
        check_slot_table(plan, cfg)
        X, y = make_data(B.CR_LOSS_SQUARED, P, rows, d, seed=21)
        W = inputs.model_matrix(K, d, seed=22)
        N, m = B.cr_plan_num_nodes(plan), B.cr_plan_load(plan)
        X_dev, y_dev, W_dev = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda(), torch.from_numpy(W).cuda()
        G = torch.zeros((K, N, m, d), device="cuda")
        ws = torch.empty(B.cr_partial_gradients_multi_workspace_bytes(plan, rows), dtype=torch.uint8, device="cuda")
        B.cr_partial_gradients_multi(plan, B.CR_LOSS_SQUARED, X_dev, y_dev, rows, W_dev, K, G, ws)
        masks = inputs.straggler_masks(cfg["n"], cfg["L"], cfg["s"], 1, seed=5)
        out = torch.zeros((1, d), device="cuda")
        for k in range(K):
            B.cr_aggregate(plan, G[k], masks, out)
            torch.cuda.synchronize()
            want = O.full_gradient(oracle_parts(B.CR_LOSS_SQUARED, X, y, W[k]))
            assert rel_l2(out[0].cpu().numpy(), want) <= REL_L2_BAR
    finally:
        B.cr_plan_destroy(plan)


def test_multi_model_rejects_bad_arguments():
    cfg = dict(n=3, L=1, s=1, P=6, d=256, code="printed_3_1")
    plan = make_plan(cfg)
    try:
        N, m = B.cr_plan_num_nodes(plan), B.cr_plan_load(plan)
        X = torch.zeros((6, 8, 256), device="cuda")
        y = torch.zeros((6, 8), device="cuda")
        W = torch.zeros((33, 256), device="cuda")
        G = torch.zeros((33, N, m, 256), device="cuda")
        ws = torch.empty(B.cr_partial_gradients_multi_workspace_bytes(plan, 8), dtype=torch.uint8, device="cuda")
        with pytest.raises(B.CodedReduceError) as e:
            B.cr_partial_gradients_multi(plan, B.CR_LOSS_SQUARED, X, y, 8, W, 33, G, ws)
        assert e.value.status == B.CR_ERR_INVALID_ARG
        with pytest.raises(B.CodedReduceError) as e:
            B.cr_partial_gradients_multi(plan, B.CR_LOSS_SQUARED, X, y, 8, W, 4, G, ws[:1024])
        assert e.value.status == B.CR_ERR_OOM
    finally:
        B.cr_plan_destroy(plan)


def test_item_order_and_ring_depth_do_not_change_results():
    """The launch order of the items and the ring depth are tuning only: every setting gives the same bits."""
    cfg = dict(n=4, L=2, s=1, P=24, d=640, code="cyclic", rows=150, K=5)
    P, d, rows, K = cfg["P"], cfg["d"], cfg["rows"], cfg["K"]
    plan = make_plan(cfg)
    try:
        X, y = make_data(B.CR_LOSS_LOGISTIC, P, rows, d, seed=31)
        W = inputs.model_matrix(K, d, seed=32)
        N, m = B.cr_plan_num_nodes(plan), B.cr_plan_load(plan)
        X_dev, y_dev, W_dev = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda(), torch.from_numpy(W).cuda()
        ws = torch.empty(B.cr_partial_gradients_multi_workspace_bytes(plan, rows), dtype=torch.uint8, device="cuda")
        ws1 = torch.empty(max(16, B.cr_partial_gradients_workspace_bytes(plan, rows)), dtype=torch.uint8, device="cuda")
        multi, single = [], []
        for order, stages in ((0, 0), (1, 2), (2, 3), (2, 4)):
            B.cr_plan_tune_items(plan, order, stages)
            G = torch.full((K, N, m, d), float("nan"), device="cuda")
            B.cr_partial_gradients_multi(plan, B.CR_LOSS_LOGISTIC, X_dev, y_dev, rows, W_dev, K, G, ws)
            G1 = torch.full((N, m, d), float("nan"), device="cuda")
            B.cr_partial_gradients_loss(plan, B.CR_LOSS_LOGISTIC, X_dev, y_dev, rows, W_dev[0], G1, ws1)
            torch.cuda.synchronize()
            B.cr_plan_device_status(plan)
            multi.append(G.cpu().numpy())
            single.append(G1.cpu().numpy())
        for g in multi[1:]:
            assert np.array_equal(g, multi[0])
        for g in single[1:]:
            assert np.array_equal(g, single[0])
        with pytest.raises(B.CodedReduceError):
            B.cr_plan_tune_items(plan, 3, 0)
        with pytest.raises(B.CodedReduceError):
            B.cr_plan_tune_items(plan, 0, 5)
    finally:
        B.cr_plan_destroy(plan)
