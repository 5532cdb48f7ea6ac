"""Host logic of the library through the C ABI (no GPU): symbol export, plan builder against the
oracle as data, schedule expansion, error codes."""
import ctypes as C
import os
import re
from itertools import combinations

import numpy as np
import pytest

from oracle import cr_oracle as O
from paper_1902_01981_b200 import binding as B
from paper_1902_01981_b200 import build as cr_build
from paper_1902_01981_b200 import inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    cr_build.build()


def host_plan(n, L, s, P=None, d=64, **kw):
    if P is None:
        P = O.partition_quantum(n, L, s)
    return B.cr_plan_create(n, L, s, P, d, device=-1, **kw)


def oracle_code(plan, kind, n, L, s):
    """The oracle's own code object for the same construction (never fed from the library)."""
    if kind == B.CR_CODE_PAPER_3_1:
        return O.Code(n, L, s, [O.printed_code_3_1()[1]] * L, kind="printed")
    if kind == B.CR_CODE_FRACTIONAL_REPETITION:
        return O.Code(n, L, s, [O.fractional_repetition_code(n, s)] * L, kind="repetition")
    raise AssertionError


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "codedreduce.h")).read()
    body = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(cr_[A-Za-z_0-9]+)\s*\(", body))
    assert {"cr_plan_create", "cr_partial_gradients", "cr_encode", "cr_decode", "cr_aggregate",
            "cr_plan_destroy"} <= declared
    lib = C.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(B._SIGNATURES), declared ^ set(B._SIGNATURES)


def test_status_strings():
    assert B.lib().cr_status_string(0) == b"CR_OK"
    assert B.lib().cr_status_string(5) == b"CR_ERR_UNDECODABLE_MASK"


@pytest.mark.parametrize("n,L,s,code", [(3, 1, 1, B.CR_CODE_PAPER_3_1), (3, 2, 1, B.CR_CODE_PAPER_3_1),
                                        (3, 4, 1, B.CR_CODE_PAPER_3_1), (4, 2, 1, B.CR_CODE_FRACTIONAL_REPETITION),
                                        (6, 2, 2, B.CR_CODE_FRACTIONAL_REPETITION)])
def test_plan_matches_oracle_for_fixed_codes(n, L, s, code):
    P = 2 * O.partition_quantum(n, L, s)
    plan = host_plan(n, L, s, P, code=code)
    try:
        oc = oracle_code(plan, code, n, L, s)
        local, _ = O.allocate(n, L, s, P, oc.B_levels)
        assert B.cr_plan_num_nodes(plan) == O.num_nodes(n, L)
        assert B.cr_plan_num_groups(plan) == O.num_groups(n, L)
        assert B.cr_plan_load(plan) == O.computation_load(n, L, s) * P
        for level in range(L):
            Bm, kappa, _ = B.cr_plan_get_B(plan, level, n)
            assert np.array_equal(Bm, oc.B_levels[level])
        for v in range(O.num_nodes(n, L)):
            part, coeff = B.cr_plan_get_slots(plan, v)
            assert [(int(p), float(c)) for p, c in zip(part, coeff)] == local[v]
        for k in range(s + 1):
            for S in combinations(range(n), k):
                mask = sum(1 << j for j in S)
                assert np.allclose(B.cr_plan_get_decode(plan, 0, mask, n), oc.decode(0, mask), atol=1e-14)
    finally:
        B.cr_plan_destroy(plan)


@pytest.mark.parametrize("n,L,s,seed", [(4, 2, 1, 0), (5, 2, 2, 0), (4, 3, 1, 5), (5, 1, 2, 2), (3, 2, 0, 0)])
def test_plan_matches_oracle_for_random_cyclic_code(n, L, s, seed):
    """Both sides draw the same SplitMix64 numbers and build B with their own arithmetic."""
    P = O.partition_quantum(n, L, s)
    plan = host_plan(n, L, s, P, code=B.CR_CODE_CYCLIC_RANDOM, seed=seed)
    try:
        B_or, sub_or = O.cyclic_random_code(n, s, seed)
        Bm, kappa, sub = B.cr_plan_get_B(plan, 0, n)
        assert sub == sub_or
        assert np.allclose(Bm, B_or, rtol=1e-12, atol=1e-13)
        assert abs(kappa - O.conditioning(B_or, s)) <= 1e-9 * kappa
        assert kappa <= 100.0
        local, _ = O.allocate(n, L, s, P, [B_or] * L)
        for v in range(O.num_nodes(n, L)):
            part, coeff = B.cr_plan_get_slots(plan, v)
            assert list(part) == [p for p, _ in local[v]]
            assert np.allclose(coeff, [c for _, c in local[v]], rtol=1e-11, atol=1e-13)
        for k in range(s + 1):
            for S in combinations(range(n), k):
                mask = sum(1 << j for j in S)
                a = B.cr_plan_get_decode(plan, L - 1, mask, n)
                assert np.allclose(a, O.decode_row(B_or, s, mask), rtol=1e-9, atol=1e-11)
                assert np.allclose(a @ Bm, 1.0, atol=1e-9)
    finally:
        B.cr_plan_destroy(plan)


@pytest.mark.parametrize("n,L,s,code", [(3, 3, 1, B.CR_CODE_PAPER_3_1), (4, 2, 1, B.CR_CODE_CYCLIC_RANDOM),
                                        (5, 2, 2, B.CR_CODE_CYCLIC_RANDOM), (4, 2, 1, B.CR_CODE_FRACTIONAL_REPETITION)])
def test_schedule_expansion_matches_oracle_walk(n, L, s, code):
    P = O.partition_quantum(n, L, s)
    plan = host_plan(n, L, s, P, code=code, seed=0)
    try:
        if code == B.CR_CODE_CYCLIC_RANDOM:
            oc = O.Code(n, L, s, [O.cyclic_random_code(n, s, 0)[0]] * L)
        else:
            oc = oracle_code(plan, code, n, L, s)
        masks = inputs.straggler_masks(n, L, s, 16, seed=3)
        for b in range(masks.shape[0]):
            nodes, layers, weights = B.cr_plan_expand(plan, masks[b])
            assert sorted(nodes.tolist()) == O.used_nodes(oc, masks[b])
            assert [O.layer_of(n, L, int(v)) for v in nodes] == layers.tolist()
            # post-order: every node appears after all used nodes of its sub-tree and its weight is the
            # decode weight its parent gives it
            seen = set()
            for v, l, w in zip(nodes.tolist(), layers.tolist(), weights.tolist()):
                i = v - O.layer_offset(n, l)             # 0-based index within the layer
                parent_group = 0 if l == 1 else O.layer_offset(n, l - 1) + i // n + 1
                a = oc.decode(l - 1, int(masks[b][parent_group]))
                assert abs(a[i % n] - w) <= 1e-9 * max(1.0, abs(w)) and w != 0.0
                if l < L:
                    kids = [O.layer_offset(n, l + 1) + n * i + j for j in range(n)]
                    a_own = oc.decode(l, int(masks[b][v + 1]))
                    assert all((k in seen) == (a_own[j] != 0.0) for j, k in enumerate(kids))
                seen.add(v)
            nbytes, used = B.cr_aggregate_bytes(plan, masks[b])
            assert used == len(nodes) and nbytes == 4 * 64 * (B.cr_plan_load(plan) * used + 1)
        nbytes, used = B.cr_aggregate_bytes(plan, masks)
        union = set()
        for b in range(masks.shape[0]):
            union |= set(O.used_nodes(oc, masks[b]))
        assert used == len(union) and nbytes == 4 * 64 * (B.cr_plan_load(plan) * used + masks.shape[0])
    finally:
        B.cr_plan_destroy(plan)


def test_integer_plans():
    plan = host_plan(3, 4, 1, code=B.CR_CODE_PAPER_3_1, dtype=B.CR_I32)
    assert B.cr_plan_int_scale(plan) == 16          # sigma = 2, L = 4
    B.cr_plan_destroy(plan)
    plan = host_plan(4, 2, 1, code=B.CR_CODE_FRACTIONAL_REPETITION, dtype=B.CR_I32)
    assert B.cr_plan_int_scale(plan) == 1
    B.cr_plan_destroy(plan)
    with pytest.raises(B.CodedReduceError) as e:
        host_plan(4, 2, 1, code=B.CR_CODE_CYCLIC_RANDOM, dtype=B.CR_I32)
    assert e.value.status == B.CR_ERR_DTYPE


def test_explicit_code():
    _, Bp = O.printed_code_3_1()
    plan = host_plan(3, 2, 1, code=B.CR_CODE_EXPLICIT, B_explicit=np.stack([Bp, Bp]))
    A, _ = O.printed_code_3_1()
    for f in range(3):
        assert np.allclose(B.cr_plan_get_decode(plan, 1, 1 << f, 3), A[f], atol=1e-13)
    B.cr_plan_destroy(plan)
    # a matrix without the span property is rejected
    bad = np.eye(3)
    with pytest.raises(B.CodedReduceError) as e:
        host_plan(3, 1, 1, P=6, code=B.CR_CODE_EXPLICIT, B_explicit=bad[None])
    assert e.value.status == B.CR_ERR_ILL_CONDITIONED


def test_error_codes():
    def status_of(**kw):
        with pytest.raises(B.CodedReduceError) as e:
            B.cr_plan_create(**kw)
        return e.value.status

    base = dict(n=4, L=2, s=1, P=24, d=64, device=-1)
    assert status_of(**{**base, "P": 40}) == B.CR_ERR_BAD_PARTITION_COUNT   # 40 is not a multiple of 24
    assert status_of(**{**base, "n": 1}) == B.CR_ERR_INVALID_ARG
    assert status_of(**{**base, "s": 4}) == B.CR_ERR_INVALID_ARG
    assert status_of(**{**base, "d": 0}) == B.CR_ERR_INVALID_ARG
    assert status_of(n=3, L=1, s=1, P=6, d=8, code=B.CR_CODE_FRACTIONAL_REPETITION, device=-1) == B.CR_ERR_CODE_UNAVAILABLE
    assert status_of(n=4, L=1, s=1, P=4, d=8, code=B.CR_CODE_PAPER_3_1, device=-1) == B.CR_ERR_CODE_UNAVAILABLE
    assert status_of(n=12, L=2, s=3, P=O.partition_quantum(12, 2, 3), d=8, max_kappa=5.0, device=-1) == B.CR_ERR_ILL_CONDITIONED
    plan = B.cr_plan_create(**base)
    try:
        groups = B.cr_plan_num_groups(plan)
        with pytest.raises(B.CodedReduceError) as e:
            B.cr_plan_expand(plan, [0b0011] + [0] * (groups - 1))
        assert e.value.status == B.CR_ERR_UNDECODABLE_MASK
        with pytest.raises(B.CodedReduceError) as e:
            B.cr_plan_expand(plan, [0b10000] + [0] * (groups - 1))
        assert e.value.status == B.CR_ERR_INVALID_ARG
        # an over-full mask below a straggling child is never consulted
        nodes, _, _ = B.cr_plan_expand(plan, [0b0001, 0b1111] + [0] * (groups - 2))
        assert 0 not in nodes.tolist()
        with pytest.raises(B.CodedReduceError) as e:
            B.cr_plan_get_decode(plan, 0, 0b0011, 4)
        assert e.value.status == B.CR_ERR_UNDECODABLE_MASK
        # device work on a host-only plan fails loudly instead of falling back
        assert B.lib().cr_encode(plan, C.c_void_p(16), C.c_void_p(16), None) == B.CR_ERR_CUDA
        assert B.lib().cr_aggregate(plan, C.c_void_p(16), C.c_void_p(16), 1, C.c_void_p(16), 0, None, 0, None) == B.CR_ERR_CUDA
    finally:
        B.cr_plan_destroy(plan)


def test_baseline_config_sizes():
    """Sizes of the five benchmark configurations (m, N, groups) follow Theorem 1."""
    for (n, L, s, P, code), (N, groups, m) in {
        (3, 1, 1, 6, B.CR_CODE_PAPER_3_1): (3, 1, 4),
        (4, 2, 1, 24, B.CR_CODE_CYCLIC_RANDOM): (20, 5, 4),
        (4, 2, 1, 48, B.CR_CODE_CYCLIC_RANDOM): (20, 5, 8),
        (5, 2, 2, 40, B.CR_CODE_CYCLIC_RANDOM): (30, 6, 9),
        (3, 4, 1, 195, B.CR_CODE_PAPER_3_1): (120, 40, 16),
    }.items():
        plan = host_plan(n, L, s, P, code=code)
        assert (B.cr_plan_num_nodes(plan), B.cr_plan_num_groups(plan), B.cr_plan_load(plan)) == (N, groups, m)
        assert B.cr_plan_load(plan) == O.computation_load(n, L, s) * P
        B.cr_plan_destroy(plan)


@pytest.mark.parametrize("n,L,s,code,batch,exactly", [(12, 2, 1, B.CR_CODE_CYCLIC_RANDOM, 64, True), (4, 3, 1, B.CR_CODE_CYCLIC_RANDOM, 40, False),
                                                      (3, 4, 1, B.CR_CODE_PAPER_3_1, 64, False), (5, 2, 2, B.CR_CODE_CYCLIC_RANDOM, 30, True),
                                                      (6, 2, 2, B.CR_CODE_FRACTIONAL_REPETITION, 16, True)])
def test_shared_message_tables_against_a_count_from_the_oracle(n, L, s, code, batch, exactly):
    """The batch kernel shares the messages of the nodes above the leaves among the patterns of a batch.
    What the host derives for that -- the union, the distinct (node, decode row) variants, the lengths of the
    full and the reduced schedules -- is recounted here from the oracle's own decode rows."""
    plan = host_plan(n, L, s, code=code)
    try:
        if code == B.CR_CODE_CYCLIC_RANDOM:
            Bm, _ = O.cyclic_random_code(n, s, 0, 100.0)
            ocode = O.Code(n, L, s, [Bm] * L, kind="solve")
        else:
            ocode = oracle_code(plan, code, n, L, s)
        masks = inputs.straggler_masks(n, L, s, batch, seed=71, exactly_s=exactly)
        used = [O.used_nodes(ocode, masks[b]) for b in range(batch)]
        union = sorted(set(v for u in used for v in u))
        lo, hi = O.layer_offset(n, L - 1), O.layer_offset(n, L)          # flat indices of layer L-1
        variants, reduced = set(), 0
        for b in range(batch):
            for v in used[b]:
                if lo <= v < hi:
                    reduced += 1
                    i = v - lo + 1                                        # node (L-1, i)
                    a = ocode.decode(L - 1, int(masks[b][O.group_of_parent(n, L - 1, i)]))
                    kids = O.children_of(n, L, L - 1, i)
                    row = tuple(np.float32(a[j]) if kids[j] in union else None for j in range(n))
                    variants.add((v, tuple(x for x in row if x is not None)))
                elif v < lo:
                    reduced += 1
        st = B.cr_plan_batch_stats(plan, masks, 2)
        assert st["entries"] == sum(len(u) for u in used)
        assert st["union"] == len(union)
        assert st["shared_nodes"] == len({v for v, _ in variants})
        assert st["variants"] == len(variants)
        assert st["reduced_entries"] == reduced
        assert st["rows"] >= st["union"]
        off = B.cr_plan_batch_stats(plan, masks, 1)
        assert off["shared_nodes"] == 0 and off["entries"] == st["entries"] and off["rows"] == off["union"]
    finally:
        B.cr_plan_destroy(plan)
