"""Batches whose patterns share sub-tree messages, pre-expanded schedules, and the bounded-wait
self-test: CUDA path against the CPU oracle through the C ABI."""
import time

import numpy as np
import pytest

from oracle import cr_oracle as O
from paper_1902_01981_b200 import binding as B
from paper_1902_01981_b200 import build as cr_build
from paper_1902_01981_b200 import inputs
from tests.gpu_common import REL_L2_BAR, check_slot_table, make_plan, rel_l2, slots_on_device

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


@pytest.fixture(scope="module", autouse=True)
def built():
    cr_build.build()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"


def tree(n, L, s, code, d, P=None, **kw):
    return dict(n=n, L=L, s=s, P=P or O.partition_quantum(n, L, s), d=d, code=code, **kw)


def aggregate(plan, G_dev, masks, d, flags=B.CR_AGG_FUSED, dtype=torch.float32):
    masks = np.asarray(masks, dtype=np.uint32).reshape(-1, B.cr_plan_num_groups(plan))
    out = torch.full((masks.shape[0], d), 7, dtype=dtype, device="cuda")
    B.cr_aggregate(plan, G_dev, masks, out, flags)
    torch.cuda.synchronize()
    assert B.cr_plan_device_status(plan) == B.CR_OK
    return out.cpu().numpy()


# ------------------------------------------------------------------ messages shared across a batch

@pytest.mark.parametrize("cfg,batch,dtype,exactly", [
    (tree(12, 2, 1, "cyclic", 4100), 64, "f32", True),        # the paper's 156-worker tree: 12 x 13 variants at most
    (tree(12, 2, 1, "cyclic", 1028), 7, "f32", False),        # few patterns, fewer than s stragglers in places
    (tree(4, 3, 1, "cyclic", 2600), 64, "f32", True),         # the 84-worker tree: messages of layer 2, replay of layer 1
    (tree(3, 4, 1, "printed_3_1", 4104), 64, "i32", False),   # deep tree, integer mode, bit-exact
    (tree(3, 4, 1, "printed_3_1", 3000), 33, "f32", False),   # odd batch (a ragged group of four), ragged tile
    (tree(5, 2, 2, "cyclic", 2052, P=80), 40, "f32", True),   # ten decode rows per node: more variants than dead rows
    (tree(6, 2, 2, "repetition", 1300), 16, "i32", True),     # 0/1 code: few children consulted, most of the union unused
    (tree(16, 2, 1, "repetition", 520), 9, "f32", False),     # widest parents
    (tree(2, 5, 1, "cyclic", 900), 12, "f32", False),         # L = 5: the eight-layer instance
    # small unions over many tiles: the form with two CTAs of eight warps per SM
    (tree(4, 2, 1, "cyclic", 77060), 16, "f32", False),
    (tree(3, 2, 1, "printed_3_1", 80004), 5, "i32", False),
    (tree(5, 2, 2, "cyclic", 76804, P=80), 12, "f32", True),
])
def test_shared_messages_match_the_oracle(cfg, batch, dtype, exactly):
    n, L, s, d = cfg["n"], cfg["L"], cfg["s"], cfg["d"]
    is_int = dtype == "i32"
    plan = make_plan(cfg, dtype=B.CR_I32 if is_int else B.CR_F32)
    try:
        code, local = check_slot_table(plan, cfg)
        G = inputs.integer_gradients(cfg["P"], d, seed=41) if is_int else inputs.partition_gradients(cfg["P"], d, seed=41)
        G_dev = slots_on_device(plan, G, torch)
        masks = inputs.straggler_masks(n, L, s, batch, seed=42, exactly_s=exactly)
        tdtype = torch.int32 if is_int else torch.float32
        B.cr_plan_tune_batch(plan, 2)                       # share whenever the tables fit
        shared = aggregate(plan, G_dev, masks, d, dtype=tdtype)
        assert B.cr_plan_last_kernel(plan) == "cr_fused_batch_tma_kernel (shared messages)"
        B.cr_plan_tune_batch(plan, 1)                       # never
        plain = aggregate(plan, G_dev, masks, d, dtype=tdtype)
        assert B.cr_plan_last_kernel(plan) == "cr_fused_batch_tma_kernel"
        # the same batch from coded gradients (one row per node)
        E = torch.zeros((B.cr_plan_num_nodes(plan), d), dtype=tdtype, device="cuda")
        B.cr_encode(plan, G_dev, E)
        B.cr_plan_tune_batch(plan, 2)
        coded = aggregate(plan, E, masks, d, B.CR_AGG_FUSED | B.CR_AGG_FROM_CODED, dtype=tdtype)
        assert B.cr_plan_last_kernel(plan) == "cr_fused_batch_tma_kernel (shared messages)"
        for b in range(batch):
            if is_int:
                want = O.execute_integer(code, local, G, masks[b])
                assert np.array_equal(shared[b].astype(np.int64), want)
                assert np.array_equal(plain[b].astype(np.int64), want)
                assert np.array_equal(coded[b].astype(np.int64), want)
            else:
                want = O.execute(code, local, G, masks[b])
                assert rel_l2(shared[b], want) <= REL_L2_BAR
                assert rel_l2(plain[b], want) <= REL_L2_BAR
                assert rel_l2(coded[b], want) <= REL_L2_BAR
    finally:
        B.cr_plan_destroy(plan)


def test_shared_messages_with_schedules_of_different_shapes():
    """A code whose decode rows consult two or three children depending on the straggler: the reduced
    schedules of one batch then differ in length and the replay takes its general form."""
    Bx = np.array([[1, 1, 0, 0], [0, 0, 1, 1], [1, 0, 2, 0], [0, 1, 0, 2]], dtype=np.float64)
    n, L, s, d = 4, 3, 1, 2200
    P = O.partition_quantum(n, L, s)
    plan = B.cr_plan_create(n, L, s, P, d, code=B.CR_CODE_EXPLICIT, B_explicit=np.stack([Bx] * L), device=0)
    try:
        code = O.Code(n, L, s, [Bx] * L, kind="solve")
        local, _ = O.allocate(n, L, s, P, code.B_levels)
        assert B.slot_partitions(plan).tolist() == [[p for p, _ in pairs] for pairs in local]
        G = inputs.partition_gradients(P, d, seed=17)
        G_dev = slots_on_device(plan, G, torch)
        masks = inputs.straggler_masks(n, L, s, 24, seed=19)
        assert len({len(B.cr_plan_expand(plan, masks[b])[0]) for b in range(24)}) > 1
        B.cr_plan_tune_batch(plan, 2)
        got = aggregate(plan, G_dev, masks, d)
        assert "shared messages" in B.cr_plan_last_kernel(plan)
        for b in range(24):
            assert rel_l2(got[b], O.execute(code, local, G, masks[b])) <= REL_L2_BAR
    finally:
        B.cr_plan_destroy(plan)


def test_built_in_choice_shares_on_wide_trees_only_when_it_pays():
    cfg = tree(12, 2, 1, "cyclic", 2048)
    plan = make_plan(cfg)
    try:
        G_dev = slots_on_device(plan, inputs.partition_gradients(cfg["P"], cfg["d"], seed=3), torch)
        aggregate(plan, G_dev, inputs.straggler_masks(12, 2, 1, 32, seed=4, exactly_s=True), cfg["d"])
        assert "shared messages" in B.cr_plan_last_kernel(plan)      # 32 x 132 entries against 12 x 13 variants
    finally:
        B.cr_plan_destroy(plan)
    cfg = tree(4, 2, 1, "cyclic", 2048)
    plan = make_plan(cfg)
    try:
        G_dev = slots_on_device(plan, inputs.partition_gradients(cfg["P"], cfg["d"], seed=3), torch)
        aggregate(plan, G_dev, inputs.straggler_masks(4, 2, 1, 3, seed=4, exactly_s=True), cfg["d"])
        assert B.cr_plan_last_kernel(plan) == "cr_fused_batch_tma_kernel"   # 3 x 12 entries: forming the variants costs more
    finally:
        B.cr_plan_destroy(plan)


# ------------------------------------------------------------------ pre-expanded schedules

@pytest.mark.parametrize("cfg,batch,dtype", [(tree(4, 2, 1, "cyclic", 4096), 1, "f32"), (tree(4, 2, 1, "cyclic", 1 << 19), 1, "f32"),
                                             (tree(12, 2, 1, "cyclic", 5004), 1, "f32"), (tree(5, 2, 2, "cyclic", 3001, P=80), 1, "f32"),
                                             (tree(3, 4, 1, "printed_3_1", 2048), 64, "i32"), (tree(12, 2, 1, "cyclic", 1500), 20, "f32"),
                                             (tree(2, 8, 0, "cyclic", 2052), 1, "f32")])
@pytest.mark.parametrize("flags", [B.CR_AGG_FUSED, B.CR_AGG_FUSED_LDG, B.CR_AGG_UNFUSED, B.CR_AGG_UNCODED_SUM])
def test_scheduled_call_equals_the_direct_call(cfg, batch, dtype, flags):
    """cr_aggregate_scheduled launches what cr_aggregate launches: same kernel, same bits; and the
    result is the oracle's.  The schedule is used twice, on different gradients."""
    n, L, s, d = cfg["n"], cfg["L"], cfg["s"], cfg["d"]
    is_int = dtype == "i32"
    tdtype = torch.int32 if is_int else torch.float32
    plan = make_plan(cfg, dtype=B.CR_I32 if is_int else B.CR_F32)
    try:
        code, local = check_slot_table(plan, cfg)
        masks = inputs.straggler_masks(n, L, s, batch, seed=52)
        sched = B.cr_schedule_create(plan, masks, flags)
        nws = B.cr_aggregate_workspace_bytes(plan, batch, flags)
        ws = torch.empty(nws, dtype=torch.uint8, device="cuda") if nws else None
        assert B.cr_schedule_bytes(sched) == B.cr_aggregate_bytes(plan, masks)
        for seed in (53, 54):
            G = inputs.integer_gradients(cfg["P"], d, seed=seed) if is_int else inputs.partition_gradients(cfg["P"], d, seed=seed)
            G_dev = slots_on_device(plan, G, torch)
            direct = torch.full((batch, d), 7, dtype=tdtype, device="cuda")
            B.cr_aggregate(plan, G_dev, masks, direct, flags, ws)
            name = B.cr_plan_last_kernel(plan)
            got = torch.full((batch, d), 9, dtype=tdtype, device="cuda")
            B.cr_aggregate_scheduled(plan, G_dev, sched, got, ws)
            torch.cuda.synchronize()
            assert B.cr_plan_last_kernel(plan) == name
            assert torch.equal(got, direct)
            if flags != B.CR_AGG_UNCODED_SUM:
                got_h = got.cpu().numpy()
                for b in range(0, batch, max(1, batch // 6)):
                    if is_int:
                        assert np.array_equal(got_h[b].astype(np.int64), O.execute_integer(code, local, G, masks[b]))
                    else:
                        assert rel_l2(got_h[b], O.execute(code, local, G, masks[b])) <= REL_L2_BAR
        assert B.cr_plan_device_status(plan) == B.CR_OK
        B.cr_schedule_destroy(sched)
    finally:
        B.cr_plan_destroy(plan)


@pytest.mark.parametrize("cfg,batch", [(tree(3, 1, 1, "printed_3_1", 1001), 1), (tree(3, 1, 1, "printed_3_1", 1001), 5),
                                       (tree(4, 2, 1, "cyclic", 3), 4), (tree(5, 1, 2, "cyclic", 1 << 16), 1),
                                       (tree(13, 2, 0, "cyclic", 2048, P=182 * 11), 1)])
def test_schedules_at_the_edges(cfg, batch):
    """Flat gradient coding (L = 1), lengths that are not multiples of four (the scalar plain-load path), a
    length of 3, a pattern of 182 consumed nodes with 11 slot rows each (a schedule too long for the kernel
    parameters, a slot count without a small divisor): scheduled call, direct call, oracle; also from coded
    gradients."""
    n, L, s, d = cfg["n"], cfg["L"], cfg["s"], cfg["d"]
    plan = make_plan(cfg)
    try:
        code, local = check_slot_table(plan, cfg)
        G = inputs.partition_gradients(cfg["P"], d, seed=81)
        G_dev = slots_on_device(plan, G, torch)
        masks = inputs.straggler_masks(n, L, s, batch, seed=82)
        E = torch.zeros((B.cr_plan_num_nodes(plan), d), device="cuda")
        B.cr_encode(plan, G_dev, E)
        for flags, src in ((B.CR_AGG_FUSED, G_dev), (B.CR_AGG_FUSED | B.CR_AGG_FROM_CODED, E)):
            sched = B.cr_schedule_create(plan, masks, flags)
            got = torch.full((batch, d), 5.0, device="cuda")
            direct = torch.full((batch, d), 6.0, device="cuda")
            B.cr_aggregate_scheduled(plan, src, sched, got)
            B.cr_aggregate(plan, src, masks, direct, flags)
            torch.cuda.synchronize()
            assert torch.equal(got, direct)
            for b in range(batch):
                assert rel_l2(got[b].cpu().numpy(), O.execute(code, local, G, masks[b])) <= REL_L2_BAR
            B.cr_schedule_destroy(sched)
        assert B.cr_plan_device_status(plan) == B.CR_OK
    finally:
        B.cr_plan_destroy(plan)


def test_schedule_errors_and_raw_pointers():
    cfg = tree(4, 2, 1, "cyclic", 1024)
    plan, other = make_plan(cfg), make_plan(cfg)
    try:
        with pytest.raises(B.CodedReduceError) as e:
            B.cr_schedule_create(plan, [0b0011, 0, 0, 0, 0])
        assert e.value.status == B.CR_ERR_UNDECODABLE_MASK
        with pytest.raises(B.CodedReduceError) as e:
            B.cr_schedule_create(plan, [0, 0, 0, 0, 0], 0x77)
        assert e.value.status == B.CR_ERR_INVALID_ARG
        code, local = check_slot_table(plan, cfg)
        G = inputs.partition_gradients(cfg["P"], cfg["d"], seed=5)
        G_dev = slots_on_device(plan, G, torch)
        masks = inputs.straggler_masks(4, 2, 1, 1, seed=6)
        sched = B.cr_schedule_create(plan, masks)
        out = torch.zeros((1, cfg["d"]), device="cuda")
        with pytest.raises(B.CodedReduceError) as e:          # a schedule serves the plan it was made for
            B.cr_aggregate_scheduled(other, G_dev, sched, out)
        assert e.value.status == B.CR_ERR_INVALID_ARG
        # plain integer addresses and a raw stream handle, as a loop that avoids the tensor look-ups passes them
        B.cr_aggregate_scheduled(plan, G_dev.data_ptr(), sched, out.data_ptr(), (0, 0), torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert rel_l2(out[0].cpu().numpy(), O.execute(code, local, G, masks[0])) <= REL_L2_BAR
        # an unfused schedule without its workspace is refused before anything is launched
        unf = B.cr_schedule_create(plan, masks, B.CR_AGG_UNFUSED)
        launches = B.cr_plan_launch_count(plan)
        with pytest.raises(B.CodedReduceError) as e:
            B.cr_aggregate_scheduled(plan, G_dev, unf, out)
        assert e.value.status == B.CR_ERR_OOM and B.cr_plan_launch_count(plan) == launches
        B.cr_schedule_destroy(unf)
        B.cr_schedule_destroy(sched)
    finally:
        B.cr_plan_destroy(plan)
        B.cr_plan_destroy(other)


# ------------------------------------------------------------------ a bounded wait that runs out

def test_a_wait_that_runs_out_sets_the_status_and_harms_nothing():
    """The kernels bound every wait and report through the plan's status word.  The self-test kernel
    waits one millisecond, through the same wait, on a barrier nobody completes: the call returns, the
    status reads CR_ERR_TIMEOUT and stays so until cleared, and the plan then works as before."""
    cfg = tree(4, 2, 1, "cyclic", 4096)
    plan = make_plan(cfg)
    try:
        code, local = check_slot_table(plan, cfg)
        G = inputs.partition_gradients(cfg["P"], cfg["d"], seed=7)
        G_dev = slots_on_device(plan, G, torch)
        masks = inputs.straggler_masks(4, 2, 1, 3, seed=8)
        assert B.cr_plan_device_status(plan) == B.CR_OK
        t0 = time.perf_counter()
        B.cr_selftest_wait(plan, 1_000_000)
        assert B.cr_plan_device_status(plan) == B.CR_ERR_TIMEOUT
        assert time.perf_counter() - t0 < 1.0
        assert B.cr_plan_device_status(plan) == B.CR_ERR_TIMEOUT        # sticky
        B.cr_plan_clear_status(plan)
        assert B.cr_plan_device_status(plan) == B.CR_OK
        for limit in (0, 10**12):
            with pytest.raises(B.CodedReduceError):
                B.cr_selftest_wait(plan, limit)
        # the production kernels take their bound the same way; a short one is still far above what a
        # healthy launch needs
        B.cr_plan_set_wait_limit(plan, 50_000_000)
        out = torch.zeros((3, cfg["d"]), device="cuda")
        B.cr_aggregate(plan, G_dev, masks, out)
        B.cr_aggregate(plan, G_dev, masks[0], out[:1])
        torch.cuda.synchronize()
        assert B.cr_plan_device_status(plan) == B.CR_OK
        assert rel_l2(out[0].cpu().numpy(), O.execute(code, local, G, masks[0])) <= REL_L2_BAR
        assert rel_l2(out[2].cpu().numpy(), O.execute(code, local, G, masks[2])) <= REL_L2_BAR
    finally:
        B.cr_plan_destroy(plan)


# ------------------------------------------------------------------ more items than a grid has rows

def test_more_nodes_than_a_grid_has_rows_of_blocks():
    """(16,4) tree without redundancy: 69904 nodes, one slot each.  The per-node and per-slot launches
    (encode, partial gradients) then exceed the 65535 rows of blocks of a grid and go in chunks."""
    n, L, s, d, rows = 16, 4, 0, 8, 2
    P = O.partition_quantum(n, L, s)
    assert P == 69904
    cfg = tree(n, L, s, "cyclic", d)
    plan = make_plan(cfg)
    try:
        code, local = check_slot_table(plan, cfg)
        N, m = B.cr_plan_num_nodes(plan), B.cr_plan_load(plan)
        assert N == 69904 and m == 1
        X, y, _ = inputs.linreg_partitions(P, rows, d, seed=61)
        w = inputs.model_vector(d, seed=62)
        G_slots = torch.full((N, m, d), float("nan"), device="cuda")
        ws = torch.empty(B.cr_partial_gradients_workspace_bytes(plan, rows), dtype=torch.uint8, device="cuda")
        B.cr_partial_gradients(plan, torch.from_numpy(X).cuda(), torch.from_numpy(y).cuda(), rows, torch.from_numpy(w).cuda(), G_slots, ws)
        torch.cuda.synchronize()
        G_parts = np.stack([O.partial_gradient_linreg(X[p], y[p], w) for p in range(P)])
        part = B.slot_partitions(plan)
        got = G_slots.cpu().numpy()
        for v in (0, 1, 65534, 65535, 65536, N - 1):
            assert rel_l2(got[v, 0], G_parts[part[v, 0]]) <= REL_L2_BAR
        assert np.isfinite(got).all()
        masks = np.zeros((1, B.cr_plan_num_groups(plan)), dtype=np.uint32)
        want = G_parts.sum(0)                                   # s = 0: the plain tree sum
        flags = B.CR_AGG_UNFUSED | B.CR_AGG_ALL_NODES
        wsu = torch.empty(B.cr_aggregate_workspace_bytes(plan, 1, flags), dtype=torch.uint8, device="cuda")
        out = torch.zeros((1, d), device="cuda")
        B.cr_aggregate(plan, G_slots, masks, out, flags, wsu)
        torch.cuda.synchronize()
        assert rel_l2(out[0].cpu().numpy(), want) <= REL_L2_BAR
        B.cr_aggregate(plan, G_slots, masks, out, B.CR_AGG_FUSED)
        torch.cuda.synchronize()
        assert rel_l2(out[0].cpu().numpy(), want) <= REL_L2_BAR
    finally:
        B.cr_plan_destroy(plan)
