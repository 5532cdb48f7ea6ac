"""Pins the CPU oracle to what the paper and plain mathematics fix, without any
reference to the CUDA path."""
from fractions import Fraction
from itertools import combinations, product
import os

import numpy as np
import pytest

from oracle import cr_oracle as O
from paper_1902_01981_b200 import inputs


# ----------------------------------------------------------------- fixtures

def _read_pairs(text):
    out = []
    for tok in text.split():
        p, c = tok.split(":")
        out.append((int(p), float(c)))
    return out


def load_example(golden_dir):
    local, message, load = {}, {}, None
    with open(os.path.join(golden_dir, "cr_example_3_2.txt")) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            if line.startswith("load"):
                load = Fraction(line.split()[1])
                continue
            head, body = line.split("|")
            kind, l, i = head.split()
            (local if kind == "local" else message)[(int(l), int(i))] = _read_pairs(body)
    return load, local, message


def load_code(golden_dir):
    A, B, w = [], [], None
    with open(os.path.join(golden_dir, "gc_code_3_1.txt")) as fh:
        for line in fh:
            t = line.split()
            if not t or t[0].startswith("#"):
                continue
            if t[0] == "A":
                A.append([float(x) for x in t[1:]])
            elif t[0] == "B":
                B.append([float(x) for x in t[1:]])
            else:
                w = [float(x) for x in t[1:]]
    return np.array(A), np.array(B), np.array(w)


def all_mask_sets(n, L, s):
    """Every assignment of a <= s straggler set to every sibling group."""
    per_group = [sum(1 << j for j in S) for k in range(s + 1) for S in combinations(range(n), k)]
    return product(per_group, repeat=O.num_groups(n, L))


def make_code(kind, n, L, s, seed=0):
    if kind == "printed":
        _, B = O.printed_code_3_1()
        return O.Code(n, L, s, [B] * L, kind="printed")
    if kind == "repetition":
        return O.Code(n, L, s, [O.fractional_repetition_code(n, s)] * L, kind="repetition")
    B, _ = O.cyclic_random_code(n, s, seed, max_kappa=100.0 if n <= 5 else 1e7)
    return O.Code(n, L, s, [B] * L, kind="solve")


# ------------------------------------------------------- load and tree sizes

def test_load_values_printed_in_the_paper():
    # Section III-B: r_CR = 4/15 for the (3,2) tree with s = 1.
    assert O.computation_load(3, 2, 1) == Fraction(4, 15)
    # Remark after Theorem 1: with n/(s+1) = 2, going from 1 to 3 layers cuts the load 7x.
    assert O.computation_load(4, 1, 1) / O.computation_load(4, 3, 1) == 7
    # L = 1 is flat gradient coding: r = (s+1)/n (Section II-C).
    assert O.computation_load(5, 1, 2) == Fraction(3, 5)
    # s = 0: every worker holds 1/N of the data.
    assert O.computation_load(3, 3, 0) == Fraction(1, O.num_nodes(3, 3))


@pytest.mark.parametrize("n,L,s", [(3, 1, 1), (3, 2, 1), (4, 2, 1), (5, 2, 2), (3, 4, 1), (4, 3, 1), (12, 2, 3)])
def test_subtree_sizes_follow_appendix_c(n, L, s):
    P = 3 * O.partition_quantum(n, L, s)
    sizes = O.subtree_sizes(n, L, s, P)
    r = O.computation_load(n, L, s)
    assert sizes[0] == Fraction(s + 1, n) * P          # Eq. rCR_proof1
    assert sizes[-1] == r * P                          # leaves hold exactly r P
    assert all(x.denominator == 1 for x in sizes)
    assert O.num_nodes(n, L) == sum(n ** l for l in range(1, L + 1))


# ----------------------------------------------------------------- GC codes

def test_printed_code_matches_the_golden_file(golden_dir):
    A_g, B_g, w = load_code(golden_dir)
    A, B = O.printed_code_3_1()
    assert np.array_equal(A, A_g) and np.array_equal(B, B_g)
    # every row of A decodes: A B = all-ones, exactly
    assert np.array_equal(A @ B, np.ones((3, 3)))
    # row f has a zero at the straggler f
    assert all(A[f, f] == 0 for f in range(3))
    # Section II-C example: g = 2 (g1/2 + g2) - (g2 - g3)
    g = np.random.default_rng(0).standard_normal((3, 7))
    assert np.allclose(w @ (B @ g), g.sum(0), atol=1e-14)


def test_least_squares_decode_reproduces_printed_rows():
    A, B = O.printed_code_3_1()
    for f in range(3):
        assert np.allclose(O.decode_row(B, 1, 1 << f), A[f], atol=1e-14)
    # no straggler: lowest two children are used
    assert np.allclose(O.decode_row(B, 1, 0), A[2], atol=1e-14)
    code = make_code("printed", 3, 2, 1)
    for mask in (0, 1, 2, 4):
        assert np.allclose(code.decode(0, mask), O.decode_row(B, 1, mask), atol=1e-14)


def test_splitmix64_known_answer():
    # First outputs of SplitMix64 from state 0 (published test vector of the
    # generator's reference implementation).
    assert O.splitmix64_stream(0, 3) == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]
    u = O.uniform_draws(7, 1000)
    assert np.all(u >= -1) and np.all(u < 1) and abs(u.mean()) < 0.1


@pytest.mark.parametrize("n,s", [(4, 1), (5, 2), (6, 2), (7, 3), (12, 3)])
def test_cyclic_code_support_and_span(n, s):
    # the kappa <= 100 screen is meant for small n; random cyclic codes get
    # ill-conditioned quickly as n and s grow, so the big cases lift it
    cap = 100.0 if n <= 5 else 1e7
    B, sub = O.cyclic_random_code(n, s, seed=3, max_kappa=cap)
    for i in range(n):
        supp = {(i + t) % n for t in range(s + 1)}
        assert {j for j in range(n) if B[i, j] != 0} == supp      # s+1 non-zeros, cyclic
        assert B[i, i] == 1.0
    ones = np.ones((1, n))
    for U in combinations(range(n), n - s):
        BU = B[list(U)]
        # all-ones lies in the row space of any n-s rows (rank test, no solver involved)
        assert np.linalg.matrix_rank(BU) == n - s
        assert np.linalg.matrix_rank(np.vstack([BU, ones])) == n - s
    for S in combinations(range(n), s):
        mask = sum(1 << j for j in S)
        a = O.decode_row(B, s, mask)
        assert all(a[j] == 0 for j in S)
        assert np.allclose(a @ B, 1.0, atol=1e-10)
    assert O.conditioning(B, s) <= cap


def test_repetition_code():
    B = O.fractional_repetition_code(4, 1)
    assert np.array_equal(B, np.array([[1, 1, 0, 0], [1, 1, 0, 0], [0, 0, 1, 1], [0, 0, 1, 1.0]]))
    for mask in (0, 1, 2, 4, 8):
        a = O.decode_row_repetition(4, 1, mask)
        assert set(a) <= {0.0, 1.0} and np.array_equal(a @ B, np.ones(4))
        assert all(a[j] == 0 for j in range(4) if mask >> j & 1)
    with pytest.raises(ValueError):
        O.fractional_repetition_code(3, 1)
    with pytest.raises(ValueError):
        O.decode_row_repetition(4, 1, 0b0011)


def test_s_zero_is_the_uncoded_tree():
    B = O.cyclic_code_from_draws(3, 0, np.zeros(0))
    assert np.array_equal(B, np.eye(3))
    code = O.Code(3, 2, 0, [B, B])
    P = O.partition_quantum(3, 2, 0)
    local, _ = O.allocate(3, 2, 0, P, code.B_levels)
    # every partition is held by exactly one node with coefficient 1
    held = sorted(p for pairs in local for p, c in pairs)
    assert held == list(range(P)) and all(c == 1.0 for pairs in local for _, c in pairs)
    G = inputs.partition_gradients(P, 33, seed=5).astype(np.float64)
    g = O.execute(code, local, G, [0] * O.num_groups(3, 2))
    assert np.allclose(g, G.sum(0), atol=1e-12)


# --------------------------------------------------------------- allocation

def test_allocation_reproduces_the_worked_example(golden_dir):
    load, local_g, message_g = load_example(golden_dir)
    _, B = O.printed_code_3_1()
    assert O.computation_load(3, 2, 1) == load
    local, subtree = O.allocate(3, 2, 1, 15, [B, B])
    for (l, i), pairs in local_g.items():
        assert local[O.flat_index(3, l, i)] == pairs
    # the message of (1,1) as a combination of partition gradients: own + subtree below
    G = np.eye(15)                                    # g_p = unit vector p
    code = O.Code(3, 2, 1, [B, B], kind="printed")
    want = np.zeros(15)
    for p, c in message_g[(1, 1)]:
        want[p] = c
    for m1 in (0, 1, 2, 4):
        masks = [0, m1, 0, 0]
        _, M = O.execute_levels(code, local, G, masks)
        assert np.allclose(M[1][0], want, atol=1e-14)
    # master with children (1,1) and (1,3): [1,0,1] gives the full gradient
    g = O.execute(code, local, G, [0b010, 0b100, 0, 0])
    assert np.allclose(g, np.ones(15), atol=1e-14)


@pytest.mark.parametrize("kind,n,L,s", [("printed", 3, 1, 1), ("printed", 3, 2, 1), ("printed", 3, 4, 1),
                                        ("solve", 4, 2, 1), ("solve", 5, 2, 2), ("solve", 4, 3, 1),
                                        ("repetition", 4, 2, 1), ("solve", 12, 2, 3)])
def test_allocation_invariants(kind, n, L, s):
    code = make_code(kind, n, L, s)
    q = O.partition_quantum(n, L, s)
    P = 2 * q if n < 12 else q
    local, subtree = O.allocate(n, L, s, P, code.B_levels)
    m = O.computation_load(n, L, s) * P
    assert all(len(pairs) == m for pairs in local)                 # equal load r P
    sizes = O.subtree_sizes(n, L, s, P)
    for v in range(O.num_nodes(n, L)):
        assert len(subtree[v]) == sizes[O.layer_of(n, L, v) - 1]
    # every partition lies in exactly s+1 layer-1 sub-trees (Appendix C)
    count = np.zeros(P, dtype=int)
    for v in range(n):
        for p in {p for p, _ in subtree[v]}:
            count[p] += 1
    assert np.all(count == s + 1)
    # a node's sub-tree set is its own set followed by what it passes down
    for v in range(O.num_nodes(n, L)):
        assert subtree[v][: int(m)] == local[v]


# ---------------------------------------------------------------- execution

@pytest.mark.parametrize("kind,n,L,s", [("printed", 3, 1, 1), ("printed", 3, 2, 1), ("solve", 4, 2, 1),
                                        ("solve", 5, 1, 2), ("repetition", 4, 2, 1), ("repetition", 4, 1, 1)])
def test_root_equals_brute_force_for_every_pattern(kind, n, L, s):
    code = make_code(kind, n, L, s)
    P = O.partition_quantum(n, L, s)
    local, subtree = O.allocate(n, L, s, P, code.B_levels)
    G = inputs.partition_gradients(P, 19, seed=11).astype(np.float64)
    want = O.full_gradient(G)
    scale = np.linalg.norm(want)
    count = 0
    for masks in all_mask_sets(n, L, s):
        g = O.execute(code, local, G, masks)
        assert np.linalg.norm(g - want) <= 1e-11 * scale
        g2, M = O.execute_levels(code, local, G, masks)
        assert np.linalg.norm(g2 - want) <= 1e-11 * scale
        # every message equals the coded gradient of its whole sub-tree set,
        # whatever the stragglers were
        for l in range(1, L + 1):
            for i in range(1, n ** l + 1):
                sub = O.coded_gradient(subtree[O.flat_index(n, l, i)], G)
                assert np.linalg.norm(M[l][i - 1] - sub) <= 1e-10 * max(1.0, np.linalg.norm(sub))
        count += 1
    assert count == sum(len(list(combinations(range(n), k))) for k in range(s + 1)) ** O.num_groups(n, L)


@pytest.mark.parametrize("kind,n,L,s", [("printed", 3, 4, 1), ("solve", 5, 2, 2), ("solve", 4, 3, 1), ("solve", 12, 2, 3)])
def test_root_equals_brute_force_random_patterns(kind, n, L, s):
    code = make_code(kind, n, L, s, seed=2)
    P = O.partition_quantum(n, L, s)
    local, _ = O.allocate(n, L, s, P, code.B_levels)
    G = inputs.partition_gradients(P, 9, seed=4).astype(np.float64)
    want = O.full_gradient(G)
    masks = inputs.straggler_masks(n, L, s, 12, seed=9)
    for b in range(masks.shape[0]):
        g = O.execute(code, local, G, masks[b])
        assert np.linalg.norm(g - want) <= 1e-9 * np.linalg.norm(want)
        used = O.used_nodes(code, masks[b])
        assert len(used) <= sum((n - s) ** l for l in range(1, L + 1))


def test_single_layer_is_flat_gradient_coding():
    # Remark after Theorem 2: L = 1 is gradient coding, g = a_f B G.
    B, _ = O.cyclic_random_code(5, 2, seed=1)
    code = O.Code(5, 1, 2, [B])
    P = O.partition_quantum(5, 1, 2)                    # = 5: one partition per chunk
    local, _ = O.allocate(5, 1, 2, P, [B])
    G = inputs.partition_gradients(P, 13, seed=2).astype(np.float64)
    for S in combinations(range(5), 2):
        mask = sum(1 << j for j in S)
        a = O.decode_row(B, 2, mask)
        assert np.allclose(O.execute(code, local, G, [mask]), a @ (B @ G), atol=1e-12)
        assert np.allclose(O.encode_all(local, G), B @ G, atol=1e-13)


def test_undecodable_pattern_is_rejected():
    code = make_code("solve", 4, 2, 1)
    P = O.partition_quantum(4, 2, 1)
    local, _ = O.allocate(4, 2, 1, P, code.B_levels)
    G = np.zeros((P, 3))
    with pytest.raises(ValueError):
        O.execute(code, local, G, [0b0011, 0, 0, 0, 0])
    # a bad mask under a straggling (unused) child is never consulted
    bad_under_straggler = [0b0001, 0b1111, 0, 0, 0]
    assert np.allclose(O.execute(code, local, G, bad_under_straggler), 0)


def test_integer_mode_is_exact():
    for kind, n, L, s in (("printed", 3, 3, 1), ("repetition", 4, 2, 1)):
        code = make_code(kind, n, L, s)
        assert O.integer_scale(code) == (2 if kind == "printed" else 1)
        P = O.partition_quantum(n, L, s)
        local, _ = O.allocate(n, L, s, P, code.B_levels)
        G = inputs.integer_gradients(P, 31, seed=3)
        want = G.astype(np.int64).sum(0)
        masks = inputs.straggler_masks(n, L, s, 10, seed=6)
        for b in range(10):
            assert np.array_equal(O.execute_integer(code, local, G, masks[b]), want)
            # dyadic coefficients: the fp64 algorithm is exact on these integers too
            assert np.array_equal(O.execute(code, local, G.astype(np.float64), masks[b]), want.astype(np.float64))


# ---------------------------------------------------------- partial gradient

def test_partial_gradient_is_the_derivative_of_the_loss():
    X, y, w_star = inputs.linreg_partitions(1, 12, 7, seed=8)
    X, y = X[0].astype(np.float64), y[0].astype(np.float64)
    w = inputs.model_vector(7, seed=9).astype(np.float64)
    g = O.partial_gradient_linreg(X, y, w)
    h = 1e-5
    for k in range(7):
        e = np.zeros(7)
        e[k] = h
        fd = (O.loss_linreg(X, y, w + e) - O.loss_linreg(X, y, w - e)) / (2 * h)
        assert abs(fd - g[k]) <= 1e-6 * max(1.0, abs(g[k]))   # quadratic loss: central difference is exact up to rounding
    # zero residual => zero gradient
    y0 = X @ w
    assert np.allclose(O.partial_gradient_linreg(X, y0, w), 0, atol=1e-12)
    assert O.normalized_error_rate(w_star, w_star) == 0.0


def test_logistic_gradient_is_the_derivative_of_the_loss():
    X, y, _ = inputs.logistic_partitions(1, 15, 6, seed=4)
    X, y = X[0].astype(np.float64), y[0].astype(np.float64)
    assert set(np.unique(y)) <= {0.0, 1.0}
    w = inputs.model_vector(6, seed=5).astype(np.float64)
    g = O.partial_gradient_logistic(X, y, w)
    h = 1e-5
    for k in range(6):
        e = np.zeros(6)
        e[k] = h
        fd = (O.loss_logistic(X, y, w + e) - O.loss_logistic(X, y, w - e)) / (2 * h)
        assert abs(fd - g[k]) <= 1e-7 * max(1.0, abs(g[k]))
    # at w = 0 every sample has probability 1/2
    assert np.allclose(O.partial_gradient_logistic(X, y, np.zeros(6)), X.T @ (0.5 - y), atol=1e-13)
    assert abs(O.loss_logistic(X, y, np.zeros(6)) - 15 * np.log(2.0)) < 1e-12


# ------------------------------------------------- planted-mistake checks

def test_pins_catch_planted_mistakes(monkeypatch):
    """A transposed B, a dropped own term or a wrong keep-rule must break a pin."""
    _, B = O.printed_code_3_1()
    code = O.Code(3, 2, 1, [B, B], kind="printed")
    G = inputs.partition_gradients(15, 5, seed=1).astype(np.float64)
    want = O.full_gradient(G)

    def root_ok():
        local, _ = O.allocate(3, 2, 1, 15, [B, B])
        return all(np.allclose(O.execute(code, local, G, m), want, atol=1e-10)
                   for m in ([0, 0, 0, 0], [1, 2, 4, 1], [4, 1, 1, 2]))

    assert root_ok()
    # transposed encoding matrix
    orig = O.comp_alloc
    monkeypatch.setattr(O, "comp_alloc", lambda Q, Bm: orig(Q, Bm.T))
    assert not root_ok()
    monkeypatch.setattr(O, "comp_alloc", orig)
    # dropped own term
    orig_cg = O.coded_gradient
    calls = {"n": 0}

    def dropped(pairs, Gp):
        calls["n"] += 1
        return orig_cg(pairs, Gp) * (0.0 if calls["n"] % 3 == 0 else 1.0)

    monkeypatch.setattr(O, "coded_gradient", dropped)
    assert not root_ok()
    monkeypatch.setattr(O, "coded_gradient", orig_cg)
    # wrong sign in a decode row
    monkeypatch.setattr(O, "printed_code_3_1", lambda: (np.array([[0, 1, 2], [1, 0, 1], [2, 1, 0.0]]), B))
    assert not root_ok()


# ------------------------------------------------ hand-worked numbers (no oracle formula repeated)

def test_conditioning_of_the_printed_code_by_hand():
    """Eq. (gc3nodes): the rows of the printed B have 1-norms 1.5, 2, 1.5; the printed decode rows
    (0,1,2), (1,0,1), (2,-1,0) then give 1*2 + 2*1.5 = 5, 1.5 + 1.5 = 3 and 2*1.5 + 1*2 = 5."""
    _, B = O.printed_code_3_1()
    assert abs(O.conditioning(B, 1) - 5.0) < 1e-12
    # doubling a row of B doubles its norm and halves its decode weight: the figure does not move
    B2 = B.copy()
    B2[1] *= 2.0
    assert abs(O.conditioning(B2, 1) - 5.0) < 1e-12
    # 0/1 repetition on (4,1): decode rows are 0/1 with two ones, every row of B has norm 2
    assert abs(O.conditioning(O.fractional_repetition_code(4, 1), 1) - 4.0) < 1e-12


def test_used_nodes_of_the_worked_example_by_hand():
    """Section III-B example on the (3,2) tree: with child 2 of the master straggling the master
    listens to (1,1) and (1,3); (1,1) with its child 3 straggling listens to (2,1), (2,2); (1,3) without
    a straggler takes its two lowest children (2,7), (2,8).  Flat indices: layer 1 = 0..2, layer 2 = 3..11."""
    code = make_code("printed", 3, 2, 1)
    assert O.used_nodes(code, [0b010, 0b100, 0, 0]) == [0, 2, 3, 4, 9, 10]
    # child 1 of the master straggles -> (1,2), (1,3); (1,2) loses its child 2 -> (2,4), (2,6);
    # (1,3) loses its child 1 -> (2,8), (2,9).  The mask below the straggler (group 1) is never read.
    assert O.used_nodes(code, [0b001, 0b111, 0b010, 0b001]) == [1, 2, 6, 8, 10, 11]


@pytest.mark.parametrize("name,count", [("cfg2", 12), ("cfg3", 12), ("cfg4", 12), ("cfg5", 30)])
def test_used_node_count_with_exactly_s_stragglers(name, count):
    """With exactly s stragglers per group a parent consults exactly n-s children, so a pattern
    consumes sum_l (n-s)^l nodes: 3+9 for the (4,2,1) and (5,2,2) trees, 2+4+8+16 for (3,4,1)."""
    from oracle import cr_setup
    cfg = inputs.CONFIGS[name]
    n, L, s = cfg["n"], cfg["L"], cfg["s"]
    code = cr_setup.code_for(cfg)
    masks = inputs.straggler_masks(n, L, s, 5, seed=21, exactly_s=True)
    for b in range(5):
        used = O.used_nodes(code, masks[b])
        assert len(used) == count == sum((n - s) ** l for l in range(1, L + 1))
        assert len(set(used)) == len(used)
        # exactly n-s of every consulted parent's children, and the master's
        assert sum(1 for v in used if v < n) == n - s


def test_linear_regression_gradient_and_loss_by_hand():
    """Eq. (g) with the squared loss on X = [[1,2],[3,4]], y = (0,1), w = (1,-1): X w = (-1,-1), residual
    (-1,-2), loss (1+4)/2, gradient X^T r = (1*-1 + 3*-2, 2*-1 + 4*-2)."""
    X = np.array([[1.0, 2.0], [3.0, 4.0]], dtype=np.float32)
    y = np.array([0.0, 1.0], dtype=np.float32)
    w = np.array([1.0, -1.0], dtype=np.float32)
    assert np.array_equal(O.partial_gradient_linreg(X, y, w), np.array([-7.0, -10.0]))
    assert O.loss_linreg(X, y, w) == 2.5
    assert O.partial_gradient_linreg(X, y, w).dtype == np.float64


def test_normalized_error_rate_by_hand():
    """Eq. (NER): w = (1,2), w* = (3,4): (4 + 4) / (9 + 16)."""
    assert O.normalized_error_rate(np.array([1.0, 2.0], dtype=np.float32), np.array([3.0, 4.0], dtype=np.float32)) == 8.0 / 25.0
    assert O.normalized_error_rate(np.zeros(2), np.array([3.0, 4.0])) == 1.0


def test_unneeded_survivor_gets_an_exact_zero():
    """CR.Execute lets a parent recover from ANY n-s children.  For B with rows (1,1,0,0), (0,0,1,1),
    (1,0,2,0), (0,1,0,2) and s = 1 the three lowest survivors are more than needed in two cases: solving
    a B_U = 1 by hand gives a = (1,1,0,0) without a straggler and with child 3 or child 4 straggling --
    the third survivor's weight is zero, so that child (and its sub-tree) is not consulted -- while
    child 1 straggling needs three children, a = (0,-1,1,1), and child 2 straggling a = (1/2,0,1/2,1/2)."""
    Bx = np.array([[1, 1, 0, 0], [0, 0, 1, 1], [1, 0, 2, 0], [0, 1, 0, 2]], dtype=np.float64)
    for mask, want in ((0b0000, [1, 1, 0, 0]), (0b1000, [1, 1, 0, 0]), (0b0100, [1, 1, 0, 0]),
                       (0b0001, [0, -1, 1, 1]), (0b0010, [0.5, 0, 0.5, 0.5])):
        a = O.decode_row(Bx, 1, mask)
        assert np.allclose(a, want, atol=1e-14)
        assert all(a[j] == 0.0 for j in range(4) if want[j] == 0)      # exact zeros, not rounding noise
        assert np.allclose(a @ Bx, 1.0, atol=1e-14)
    code = O.Code(4, 2, 1, [Bx, Bx], kind="solve")
    # master without straggler: children 1, 2 only; each of them, without straggler, its children 1, 2
    assert O.used_nodes(code, [0, 0, 0, 0, 0]) == [0, 1, 4, 5, 8, 9]
    # child 1 of the master straggles: children 2, 3, 4 are all needed
    assert sorted(v for v in O.used_nodes(code, [1, 0, 0, 0, 0]) if v < 4) == [1, 2, 3]
