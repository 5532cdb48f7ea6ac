"""The benchmark configurations at their full sizes, in the launch shapes bench.py times.

Aggregation-only configurations compare sampled output columns (both tile edges plus a random
spread) with the oracle, which computes any column independently of the others; the two
linear-regression configurations run their whole gradient-descent loops.
"""
import numpy as np
import pytest

from oracle import cr_oracle as O
from oracle import cr_setup
from paper_1902_01981_b200 import binding as B
from paper_1902_01981_b200 import build as cr_build
from paper_1902_01981_b200 import inputs
from tests.gpu_common import REL_L2_BAR, check_slot_table, make_plan, rel_l2, slots_on_device

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


@pytest.fixture(scope="module", autouse=True)
def built():
    cr_build.build()
    assert torch.cuda.is_available()


def sample_columns(d, seed=0, edge=600, spread=3000):
    rng = np.random.default_rng(seed)
    cols = np.concatenate([np.arange(min(edge, d)), np.arange(max(0, d - edge), d), rng.integers(0, d, spread)])
    return np.unique(cols)


def aggregate_full(cfg, dtype, iters, flags=B.CR_AGG_FUSED):
    """Runs `iters` cr_aggregate calls of a full-size configuration; yields per call the sampled
    GPU columns, the matching partition-gradient columns and the masks."""
    is_int = dtype == B.CR_I32
    plan = make_plan(cfg, dtype=dtype)
    try:
        code, local = check_slot_table(plan, cfg)
        d, batch = cfg["d"], cfg.get("batch", 1)
        G = (inputs.integer_gradients(cfg["P"], d, cfg["seed"], cfg["int_bound"]) if is_int
             else inputs.partition_gradients(cfg["P"], d, cfg["seed"], cfg.get("std", 1.0)))
        G_dev = slots_on_device(plan, G, torch)
        cols = sample_columns(d)
        cols_dev = torch.from_numpy(cols).cuda()
        G_cols = np.ascontiguousarray(G[:, cols])
        del G
        masks = inputs.straggler_masks(cfg["n"], cfg["L"], cfg["s"], iters * batch, cfg["mask_seed"],
                                       cfg.get("exactly_s", False)).reshape(iters, batch, -1)
        out = torch.zeros((batch, d), dtype=torch.int32 if is_int else torch.float32, device="cuda")
        for it in range(iters):
            out.fill_(3)
            B.cr_aggregate(plan, G_dev, masks[it], out, flags)
            torch.cuda.synchronize()
            yield code, local, out.index_select(1, cols_dev).cpu().numpy(), G_cols, masks[it]
        assert B.cr_plan_device_status(plan) == B.CR_OK
    finally:
        B.cr_plan_destroy(plan)


def test_cfg2_aggregation_d_2_20():
    cfg = inputs.CONFIGS["cfg2"]
    for it, (code, local, got, G_cols, masks) in enumerate(aggregate_full(cfg, B.CR_F32, cfg["iters"])):
        want = O.execute(code, local, G_cols, masks[0]) if it % 10 == 0 else O.full_gradient(G_cols)
        assert rel_l2(got[0], want) <= REL_L2_BAR


def test_cfg4_large_gradient_d_2_24():
    cfg = inputs.CONFIGS["cfg4"]
    for it, (code, local, got, G_cols, masks) in enumerate(aggregate_full(cfg, B.CR_F32, cfg["iters"])):
        assert bin(int(masks[0][0])).count("1") == 2
        assert rel_l2(got[0], O.execute(code, local, G_cols, masks[0])) <= REL_L2_BAR
        assert rel_l2(got[0], O.full_gradient(G_cols)) <= REL_L2_BAR


def test_cfg5_deep_tree_batch_fp32():
    cfg = inputs.CONFIGS["cfg5"]
    for it, (code, local, got, G_cols, masks) in enumerate(aggregate_full(cfg, B.CR_F32, 2)):
        want_sum = O.full_gradient(G_cols)
        for b in range(cfg["batch"]):
            assert rel_l2(got[b], want_sum) <= REL_L2_BAR
        for b in range(0, cfg["batch"], 16):
            assert rel_l2(got[b], O.execute(code, local, G_cols, masks[b])) <= REL_L2_BAR


def test_cfg5_deep_tree_batch_int32_bit_exact():
    cfg = inputs.CONFIGS["cfg5"]
    for it, (code, local, got, G_cols, masks) in enumerate(aggregate_full(cfg, B.CR_I32, 2)):
        want = G_cols.astype(np.int64).sum(0)
        for b in range(cfg["batch"]):
            assert np.array_equal(got[b].astype(np.int64), want)
        assert np.array_equal(O.execute_integer(code, local, G_cols, masks[0]), want)


@pytest.mark.parametrize("name", ["cfg_tree12", "cfg_tree43"])
def test_paper_cluster_trees_d_2_22(name):
    """The (12,2) and (4,3) trees of the paper's 156- and 84-worker clusters at d = 2^22."""
    cfg = inputs.CONFIGS[name]
    for it, (code, local, got, G_cols, masks) in enumerate(aggregate_full(cfg, B.CR_F32, 4)):
        assert rel_l2(got[0], O.execute(code, local, G_cols, masks[0])) <= REL_L2_BAR
        assert rel_l2(got[0], O.full_gradient(G_cols)) <= REL_L2_BAR


@pytest.mark.parametrize("name", ["cfg_tree12", "cfg_tree43"])
def test_paper_cluster_trees_batches_of_64_d_2_20(name):
    """Batches of 64 patterns on the paper's trees at d = 2^20, as `bench.py --batch 64 --d 1048576` times
    them: the patterns share the messages of the layer above the leaves.  Every pattern against the plain
    sum, a spread of them against CR.Execute."""
    cfg = dict(inputs.CONFIGS[name], d=1 << 20, batch=64)
    for code, local, got, G_cols, masks in aggregate_full(cfg, B.CR_F32, 2):
        want_sum = O.full_gradient(G_cols)
        for b in range(64):
            assert rel_l2(got[b], want_sum) <= REL_L2_BAR
        for b in range(0, 64, 9):
            assert rel_l2(got[b], O.execute(code, local, G_cols, masks[b])) <= REL_L2_BAR


@pytest.mark.parametrize("n,s,code", [(12, 1, "cyclic"), (12, 3, "repetition"), (3, 1, "printed_3_1")])
def test_flat_gradient_coding_d_2_22(n, s, code):
    """L = 1: CodedReduce is flat gradient coding (master and n workers, m = s + 1 slot rows per worker).
    Full-size single patterns, as `bench.py --tree n,1,s,code --d 4194304` launches them, and a batch of
    patterns over the same slots; the result is the plain sum of the partition gradients."""
    cfg = dict(n=n, L=1, s=s, P=O.partition_quantum(n, 1, s), d=1 << 22, code=code, seed=5, mask_seed=6, batch=1,
               exactly_s=True, std=1.0)
    for code_, local, got, G_cols, masks in aggregate_full(cfg, B.CR_F32, 3):
        assert rel_l2(got[0], O.execute(code_, local, G_cols, masks[0])) <= REL_L2_BAR
        assert rel_l2(got[0], O.full_gradient(G_cols)) <= REL_L2_BAR
    for code_, local, got, G_cols, masks in aggregate_full(dict(cfg, batch=6, exactly_s=False), B.CR_F32, 1):
        for b in range(6):
            assert rel_l2(got[b], O.execute(code_, local, G_cols, masks[b])) <= REL_L2_BAR


@pytest.mark.parametrize("s", [1, 2, 3, 5])
@pytest.mark.parametrize("d", [5001, 6500, 120000])
def test_paper_cluster_straggler_fractions(s, d):
    """(12,2) tree with s = alpha n stragglers tolerated per group for the paper's alpha = 1/12 .. 5/12, at
    the model sizes of its three experiments (p = 5001, 6500, ~1.2e5); (s+1) divides 12, so the 0/1
    fractional repetition code exists for each (m = (s+1)^2 slots per node, up to 36)."""
    cfg = dict(n=12, L=2, s=s, P=O.partition_quantum(12, 2, s), d=d, code="repetition", seed=3, mask_seed=4,
               int_bound=1 << 10)
    for dtype in (B.CR_F32, B.CR_I32):
        for flags in (B.CR_AGG_FUSED, B.CR_AGG_FUSED_LDG):
            for code, local, got, G_cols, masks in aggregate_full(dict(cfg, batch=1), dtype, 2, flags):
                if dtype == B.CR_I32:
                    assert np.array_equal(got[0].astype(np.int64), G_cols.astype(np.int64).sum(0))
                else:
                    assert rel_l2(got[0], O.execute(code, local, G_cols, masks[0])) <= REL_L2_BAR
    # a batch of patterns through the batch kernel
    for code, local, got, G_cols, masks in aggregate_full(dict(cfg, batch=5), B.CR_F32, 1):
        for b in range(5):
            assert rel_l2(got[b], O.execute(code, local, G_cols, masks[b])) <= REL_L2_BAR


@pytest.mark.parametrize("dtype", [B.CR_F32, B.CR_I32])
def test_repetition_code_d_2_20(dtype):
    cfg = inputs.CONFIGS["cfg_rep"]
    for it, (code, local, got, G_cols, masks) in enumerate(aggregate_full(cfg, dtype, cfg["iters"])):
        if dtype == B.CR_I32:
            assert np.array_equal(got[0].astype(np.int64), G_cols.astype(np.int64).sum(0))
        else:
            assert rel_l2(got[0], O.execute(code, local, G_cols, masks[0])) <= REL_L2_BAR


# --------------------------------------------------------------------------- gradient-descent loops

def gd_loop(cfg, mask_sets, w0, lr_eff):
    """Partial gradients -> aggregate -> w -= lr_eff * g on the GPU; the oracle is evaluated at the
    GPU's w_t (gradient parity) and also runs freely from the same start (loss trajectory)."""
    n, L, s, P, d, rows = cfg["n"], cfg["L"], cfg["s"], cfg["P"], cfg["d"], cfg["rows"]
    plan = make_plan(cfg)
    try:
        code, local = check_slot_table(plan, cfg)
        X, y, w_star = inputs.linreg_partitions(P, rows, d, cfg["seed"], cfg["x_std"], cfg["noise_std"])
        X64, y64 = X.astype(np.float64), y.astype(np.float64)
        N, m = B.cr_plan_num_nodes(plan), B.cr_plan_load(plan)
        X_dev, y_dev = torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda()
        w_dev = torch.from_numpy(w0.copy()).cuda()
        G_slots = torch.zeros((N, m, d), device="cuda")
        ws = torch.empty(B.cr_partial_gradients_workspace_bytes(plan, rows), dtype=torch.uint8, device="cuda")
        out = torch.zeros((len(mask_sets[0]), d), device="cuda")

        def oracle_parts(w):
            return np.stack([O.partial_gradient_linreg(X64[p], y64[p], w) for p in range(P)])

        def total_loss(w):
            return sum(O.loss_linreg(X64[p], y64[p], w) for p in range(P))

        w_free = w0.astype(np.float64)
        losses_gpu, losses_free, ner = [], [], []
        for t, masks in enumerate(mask_sets):
            w_t = w_dev.cpu().numpy()
            B.cr_partial_gradients(plan, X_dev, y_dev, rows, w_dev, G_slots, ws)
            B.cr_aggregate(plan, G_slots, masks, out)
            torch.cuda.synchronize()
            got = out.cpu().numpy()
            if t < 3 or t % 7 == 0 or t == len(mask_sets) - 1:
                parts = oracle_parts(w_t)                       # oracle at the GPU's own iterate
                g_def = O.full_gradient(parts)
                for b in range(len(masks)):
                    assert rel_l2(got[b], O.execute(code, local, parts, masks[b])) <= REL_L2_BAR, (t, b)
                    assert rel_l2(got[b], g_def) <= REL_L2_BAR
            for b in range(1, len(masks)):                      # every straggler pattern gives the same gradient
                assert rel_l2(got[b], got[0]) <= 2 * REL_L2_BAR
            losses_gpu.append(total_loss(w_t))
            losses_free.append(total_loss(w_free))
            ner.append(O.normalized_error_rate(w_t, w_star))
            w_dev -= lr_eff * out[0]
            w_free = w_free - lr_eff * O.execute(code, local, oracle_parts(w_free), masks[0])
        assert B.cr_plan_device_status(plan) == B.CR_OK
        return np.array(losses_gpu), np.array(losses_free), np.array(ner)
    finally:
        B.cr_plan_destroy(plan)


def test_cfg1_tiny_tree_linear_regression_loop():
    cfg = inputs.CONFIGS["cfg1"]
    masks = [np.array([[0], [1], [2], [4]], dtype=np.uint32)] * cfg["iters"]      # none, and each single straggler
    w0 = inputs.model_vector(cfg["d"], seed=1)
    lg, lf, ner = gd_loop(cfg, masks, w0, cfg["lr"])
    assert np.all(np.abs(lg - lf) <= 1e-4 * lf)
    assert np.all(np.diff(lg) < 0) and np.all(np.diff(ner) < 0)


def test_cfg3_end_to_end_linear_regression_loop():
    cfg = inputs.CONFIGS["cfg3"]
    mk = inputs.straggler_masks(cfg["n"], cfg["L"], cfg["s"], cfg["iters"], cfg["mask_seed"])
    w0 = np.zeros(cfg["d"], dtype=np.float32)
    lg, lf, ner = gd_loop(cfg, [mk[t:t + 1] for t in range(cfg["iters"])], w0, cfg["lr"] / cfg["P"])
    assert np.all(np.abs(lg - lf) <= 1e-4 * lf)
    assert np.all(np.diff(lg) < 0) and np.all(np.diff(ner) < 0)
    assert lg[-1] < 0.1 * lg[0]


# --------------------------------------------------------------------------- degenerate shapes

@pytest.mark.parametrize("d", [1, 3, 4, 255, 256, 257, 1020])
@pytest.mark.parametrize("flags", [B.CR_AGG_FUSED, B.CR_AGG_FUSED_LDG, B.CR_AGG_UNFUSED])
def test_small_and_ragged_lengths(d, flags):
    cfg = dict(n=3, L=2, s=1, P=15, d=d, code="printed_3_1")
    plan = make_plan(cfg)
    try:
        code, local = check_slot_table(plan, cfg)
        G = inputs.partition_gradients(15, d, seed=d)
        G_dev = slots_on_device(plan, G, torch)
        masks = inputs.straggler_masks(3, 2, 1, 5, seed=1)
        ws = None
        nbytes = B.cr_aggregate_workspace_bytes(plan, 5, flags)
        if nbytes:
            ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        out = torch.zeros((5, d), device="cuda")
        B.cr_aggregate(plan, G_dev, masks, out, flags, ws)
        one = torch.zeros((1, d), device="cuda")
        B.cr_aggregate(plan, G_dev, masks[2], one, flags, ws)
        torch.cuda.synchronize()
        for b in range(5):
            assert rel_l2(out[b].cpu().numpy(), O.execute(code, local, G, masks[b])) <= REL_L2_BAR
        assert rel_l2(one[0].cpu().numpy(), O.execute(code, local, G, masks[2])) <= REL_L2_BAR
        with pytest.raises(B.CodedReduceError):
            B.cr_aggregate(plan, G_dev, np.zeros((0, 4), dtype=np.uint32), out, flags, ws)    # empty batch
    finally:
        B.cr_plan_destroy(plan)


def test_unaligned_buffers_take_the_plain_load_path():
    cfg = dict(n=4, L=2, s=1, P=24, d=1024, code="cyclic")
    plan = make_plan(cfg)
    try:
        code, local = check_slot_table(plan, cfg)
        G = inputs.partition_gradients(24, 1024, seed=5)
        base = torch.zeros(20 * 4 * 1024 + 1, device="cuda")
        G_dev = base[1:].view(20, 4, 1024)                       # 4-byte aligned only
        G_dev.copy_(slots_on_device(plan, G, torch))
        masks = inputs.straggler_masks(4, 2, 1, 1, seed=1)
        out = torch.zeros((1, 1024), device="cuda")
        B.cr_aggregate(plan, G_dev, masks, out)
        torch.cuda.synchronize()
        assert rel_l2(out[0].cpu().numpy(), O.execute(code, local, G, masks[0])) <= REL_L2_BAR
    finally:
        B.cr_plan_destroy(plan)
