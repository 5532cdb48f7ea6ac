"""CodedReduce oracle -- TEST INFRASTRUCTURE, not product code.

A plain, slow, fp64 CPU restatement of the coded tree aggregation of CodedReduce
(CR), written from the paper.  It exists so that tests, the smoke check and the
benchmark's CPU-baseline leg have something independent to compare the CUDA path
with.  Nothing in the product package may import or call it, and it imports
nothing from the product package.

Indexing used throughout (0-based restatement of Section III-A):
  * layers l = 1..L hold n**l worker nodes; the master is layer 0.
  * node (l, i), i = 1..n**l, has flat index  offset(l) + i - 1  with
    offset(l) = n + n**2 + ... + n**(l-1);  its children are
    (l+1, n(i-1)+1 .. n i)                                   (Algorithm 2).
  * a "group" is the n children of one parent.  Group 0 belongs to the master;
    the group of the children of flat node v is  v + 1.
  * a straggler mask is an integer whose bit j (0-based) marks child j of that
    group as a straggler.

Parity status of each function is given in its docstring ("pinned by ...");
the only unpinned choice is which decode row is used when fewer than s children
straggle (any valid row gives the same gradient; see `survivors`).
"""
from __future__ import annotations

from fractions import Fraction
from itertools import combinations

import numpy as np

# --------------------------------------------------------------------------
# Tree indexing (Section III-A, definition of the (n, L)-regular tree)
# --------------------------------------------------------------------------


def num_nodes(n: int, L: int) -> int:
    """N = n + n**2 + ... + n**L workers (Section III-A)."""
    return sum(n ** l for l in range(1, L + 1))


def num_groups(n: int, L: int) -> int:
    """One sibling group per parent, master included: 1 + n + ... + n**(L-1)."""
    return sum(n ** l for l in range(0, L))


def layer_offset(n: int, l: int) -> int:
    return sum(n ** t for t in range(1, l))


def flat_index(n: int, l: int, i: int) -> int:
    """Flat index of node (l, i), l >= 1, i = 1..n**l."""
    assert 1 <= i <= n ** l
    return layer_offset(n, l) + i - 1


def layer_of(n: int, L: int, v: int) -> int:
    for l in range(1, L + 1):
        if v < layer_offset(n, l) + n ** l:
            return l
    raise ValueError("node index out of range")


def children_of(n: int, L: int, l: int, i: int) -> list[int]:
    """Flat indices of the children of (l, i); (0, 1) is the master."""
    assert l < L
    return [flat_index(n, l + 1, n * (i - 1) + j) for j in range(1, n + 1)]


def group_of_parent(n: int, l: int, i: int) -> int:
    """Index of the sibling group formed by the children of (l, i)."""
    return 0 if l == 0 else flat_index(n, l, i) + 1


# --------------------------------------------------------------------------
# Computation load (Theorem 1, Eq. rCR_lemma; Appendix C recursion)
# --------------------------------------------------------------------------


def computation_load(n: int, L: int, s: int) -> Fraction:
    """r_CR = 1 / sum_{l=1..L} (n/(s+1))**l  (Theorem 1).

    Pinned by the values the paper prints: 4/15 for (3,2), s=1, and the 7x
    reduction from L=1 to L=3 when n/(s+1) = 2.
    """
    q = Fraction(n, s + 1)
    return 1 / sum(q ** l for l in range(1, L + 1))


def subtree_sizes(n: int, L: int, s: int, P: int) -> list[Fraction]:
    """|D^{T(l,.)}| for l = 1..L in atomic partitions (Appendix C, achievability).

    |D^{T(1,i)}| = (s+1)/n * P and every layer keeps r*P before passing the rest
    through another (s+1)/n redundant split.
    """
    rho = Fraction(s + 1, n)
    r = computation_load(n, L, s)
    sizes = [rho * P]
    for _ in range(2, L + 1):
        sizes.append(rho * (sizes[-1] - r * P))
    return sizes


def partition_quantum(n: int, L: int, s: int) -> int:
    """Smallest P for which every cut of the allocation is an integer.

    The paper says "uniformly partition" and is silent when sizes do not divide;
    the reading used here is to require P to be a multiple of
    sum_l n**l (s+1)**(L-l), which makes r*P = c (s+1)**L and every chunk whole.
    """
    return sum(n ** l * (s + 1) ** (L - l) for l in range(1, L + 1))


# --------------------------------------------------------------------------
# Gradient-coding matrices (Section II-C; Eq. gc3nodes)
# --------------------------------------------------------------------------


def printed_code_3_1():
    """(A, B) exactly as printed in Eq. gc3nodes for n = 3, s = 1.

    Row f of A is the decode row when child f straggles.
    """
    A = np.array([[0.0, 1.0, 2.0], [1.0, 0.0, 1.0], [2.0, -1.0, 0.0]])
    B = np.array([[0.5, 1.0, 0.0], [0.0, 1.0, -1.0], [0.5, 0.0, 1.0]])
    return A, B


def splitmix64_stream(seed: int, count: int) -> list[int]:
    """`count` outputs of the SplitMix64 generator (Steele, Lea, Flood 2014)
    started from state `seed`.  Counter based: output k depends only on
    seed + (k+1) * golden-gamma."""
    mask = (1 << 64) - 1
    out = []
    state = seed & mask
    for _ in range(count):
        state = (state + 0x9E3779B97F4A7C15) & mask
        z = state
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & mask
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & mask
        z = z ^ (z >> 31)
        out.append(z)
    return out


def uniform_draws(seed: int, count: int) -> np.ndarray:
    """Uniform numbers in [-1, 1): the top 53 bits of each SplitMix64 output
    give u = bits / 2**53, mapped to 2u - 1 (every step exact in fp64)."""
    raw = splitmix64_stream(seed, count)
    return np.array([2.0 * ((z >> 11) / 9007199254740992.0) - 1.0 for z in raw])


def cyclic_code_from_draws(n: int, s: int, draws: np.ndarray) -> np.ndarray:
    """Encoding matrix B (n x n) with cyclic support from s*(n-1) random numbers.

    The paper defers the construction of B to the gradient-coding paper it
    cites; the property it needs is that each row has s+1 non-zeros and that any
    n-s rows span the all-ones vector (Section II-C).  Construction used:
    take H (s x n) whose first n-1 columns are the draws (row-major) and whose
    last column makes every row of H sum to zero; row i of B is supported on
    {i, i+1, .., i+s} mod n, has b_ii = 1, and lies in the null space of H.
    null(H) has dimension n-s and contains the all-ones vector, so any n-s
    independent rows of B span it.

    Pinned by: support pattern, H B^T = 0, and the rank test over every
    (n-s)-subset in the tests.
    """
    B = np.zeros((n, n))
    if s == 0:
        return np.eye(n)
    H = np.zeros((s, n))
    H[:, : n - 1] = np.asarray(draws, dtype=np.float64).reshape(s, n - 1)
    H[:, n - 1] = -H[:, : n - 1].sum(axis=1)
    for i in range(n):
        others = [(i + t) % n for t in range(1, s + 1)]
        x = np.linalg.solve(H[:, others], -H[:, i])
        B[i, i] = 1.0
        for col, val in zip(others, x):
            B[i, col] = val
    return B


def fractional_repetition_code(n: int, s: int) -> np.ndarray:
    """0/1 fractional-repetition B: children form n/(s+1) blocks of s+1
    identical rows; block q covers data chunks q(s+1) .. q(s+1)+s.
    Exists only when (s+1) divides n."""
    if n % (s + 1) != 0:
        raise ValueError("fractional repetition needs (s+1) | n")
    B = np.zeros((n, n))
    for i in range(n):
        q = i // (s + 1)
        B[i, q * (s + 1): (q + 1) * (s + 1)] = 1.0
    return B


def survivors(n: int, s: int, straggler_mask: int) -> list[int]:
    """The n-s children a parent decodes from: the lowest-indexed
    non-stragglers.  (The paper indexes decode rows by exactly-s straggler sets;
    with fewer stragglers any n-s survivors work and give the same result in
    exact arithmetic -- this choice is a convention, unpinned by the paper.)"""
    if bin(straggler_mask).count("1") > s:
        raise ValueError("more than s stragglers in a sibling group: not decodable")
    alive = [j for j in range(n) if not (straggler_mask >> j) & 1]
    return alive[: n - s]


def decode_row(B: np.ndarray, s: int, straggler_mask: int) -> np.ndarray:
    """Decode row a (length n): supported on `survivors`, with a B = all-ones
    (Section II-C: g = a_f B G).  Solved by least squares on the consistent
    system B_U^T a_U = 1.

    A survivor whose weight comes out of the solver as rounding noise (at most
    1e-13 of the largest weight) gets an exact zero: the parent needs "any n-s"
    children, and a child with zero weight is one it does not consult.

    Pinned by the printed A for the printed B, by a B = 1 residuals, by the
    root-equals-brute-force tests, and (the zeroing rule) by a 4 x 4 code whose
    decode rows are solved by hand.
    """
    n = B.shape[0]
    U = survivors(n, s, straggler_mask)
    a_U, *_ = np.linalg.lstsq(B[U, :].T, np.ones(n), rcond=None)
    # a survivor that is not needed comes out of the solver as rounding noise: that is a zero
    a_U[np.abs(a_U) <= 1e-13 * np.max(np.abs(a_U))] = 0.0
    a = np.zeros(n)
    a[U] = a_U
    return a


def decode_row_repetition(n: int, s: int, straggler_mask: int) -> np.ndarray:
    """0/1 decode row for the fractional-repetition code: weight 1 on the
    lowest-indexed non-straggler of every block of s+1 identical children."""
    if bin(straggler_mask).count("1") > s:
        raise ValueError("more than s stragglers in a sibling group: not decodable")
    a = np.zeros(n)
    for q in range(n // (s + 1)):
        block = range(q * (s + 1), (q + 1) * (s + 1))
        first = next(j for j in block if not (straggler_mask >> j) & 1)
        a[first] = 1.0
    return a


def conditioning(B: np.ndarray, s: int) -> float:
    """kappa = max over exactly-s straggler sets of sum_j |a_j| * ||b_j||_1:
    the worst-case amplification of rounding error by one decode.
    Pinned by the hand value 5 for the code printed in Eq. gc3nodes (row norms
    1.5, 2, 1.5 against the printed decode rows) and by its invariance under
    rescaling a row of B."""
    n = B.shape[0]
    worst = 0.0
    for S in combinations(range(n), s):
        mask = sum(1 << j for j in S)
        a = decode_row(B, s, mask)
        worst = max(worst, float(np.sum(np.abs(a) * np.abs(B).sum(axis=1))))
    return worst


def cyclic_random_code(n: int, s: int, seed: int, max_kappa: float = 100.0, tries: int = 64):
    """Draw cyclic codes from sub-seeds seed, seed+1, .. until kappa <= max_kappa.
    Returns (B, sub_seed)."""
    for t in range(tries):
        B = cyclic_code_from_draws(n, s, uniform_draws(seed + t, s * (n - 1)))
        if conditioning(B, s) <= max_kappa:
            return B, seed + t
    raise ValueError("no well-conditioned code found")


# --------------------------------------------------------------------------
# CompAlloc (Algorithm 1) and CR.Allocate (Algorithm 2, first procedure)
# --------------------------------------------------------------------------


def comp_alloc(Q: list, B: np.ndarray) -> list[list]:
    """CompAlloc(D, B): cut the list Q of (partition, coefficient) pairs into
    k = n consecutive equal chunks D_1..D_k; child i receives the union over
    kappa of b_{i kappa} D_kappa, i.e. every pair of chunk kappa with its
    coefficient multiplied by b_{i kappa}, chunks taken in increasing kappa."""
    n = B.shape[0]
    assert len(Q) % n == 0, "data set does not split uniformly"
    size = len(Q) // n
    chunks = [Q[k * size: (k + 1) * size] for k in range(n)]
    out = []
    for i in range(n):
        mine = []
        for k in range(n):
            if B[i, k] != 0.0:
                mine.extend((p, c * B[i, k]) for (p, c) in chunks[k])
        out.append(mine)
    return out


def allocate(n: int, L: int, s: int, P: int, B_levels: list[np.ndarray]):
    """CR.Allocate.  B_levels[l-1] is the encoding matrix used when the parents
    at layer l-1 split their pass-down set among their layer-l children (the
    paper uses one B for all layers; a list of identical matrices expresses that).

    Returns (local, subtree): local[v] = D(l,i) and subtree[v] = D^{T(l,i)},
    each a list of (partition, coefficient) pairs, v the flat node index.
    Every node keeps the FIRST r*P pairs of its sub-tree's set (the worked
    example keeps "the first two sub-sets") and passes the rest down.
    """
    rP = computation_load(n, L, s) * P
    assert rP.denominator == 1, "r_CR * P must be an integer"
    m = int(rP)
    N = num_nodes(n, L)
    local = [None] * N
    subtree = [None] * N
    passdown = {(0, 1): [(p, 1.0) for p in range(P)]}
    for l in range(1, L + 1):
        for i in range(1, n ** (l - 1) + 1):
            parts = comp_alloc(passdown[(l - 1, i)], B_levels[l - 1])
            for j in range(1, n + 1):
                subtree[flat_index(n, l, n * (i - 1) + j)] = parts[j - 1]
        for i in range(1, n ** l + 1):
            v = flat_index(n, l, i)
            local[v] = subtree[v][:m]
            passdown[(l, i)] = subtree[v][m:]
    for i in range(1, n ** L + 1):
        assert not passdown[(L, i)], "leaves must keep their whole set"
    return local, subtree


# --------------------------------------------------------------------------
# CR.Execute (Algorithm 2, second procedure)
# --------------------------------------------------------------------------


def coded_gradient(pairs: list, G_parts: np.ndarray) -> np.ndarray:
    """g_{D(l,i)} = sum over the node's (partition, coefficient) pairs of
    coefficient * g_partition  (scaled data sets, Section III-A)."""
    e = np.zeros(G_parts.shape[1], dtype=np.float64)
    for p, c in pairs:
        e += c * G_parts[p].astype(np.float64)
    return e


def encode_all(local: list, G_parts: np.ndarray) -> np.ndarray:
    return np.stack([coded_gradient(pairs, G_parts) for pairs in local])


class Code:
    """A per-level list of encoding matrices plus the rule that yields decode
    rows.  kind is 'solve' (least squares on the survivors), 'printed'
    (rows of the printed A of Eq. gc3nodes) or 'repetition' (0/1 rows)."""

    def __init__(self, n, L, s, B_levels, kind="solve"):
        self.n, self.L, self.s, self.kind = n, L, s, kind
        self.B_levels = [np.asarray(B, dtype=np.float64) for B in B_levels]
        assert len(self.B_levels) == L

    def decode(self, parent_layer: int, straggler_mask: int) -> np.ndarray:
        """Decode row used by a parent at `parent_layer` (0 = master)."""
        B = self.B_levels[parent_layer]
        if self.kind == "repetition":
            return decode_row_repetition(self.n, self.s, straggler_mask)
        if self.kind == "printed":
            A, _ = printed_code_3_1()
            if bin(straggler_mask).count("1") > 1:
                raise ValueError("more than s stragglers in a sibling group: not decodable")
            # no straggler: decode from the two lowest-indexed children, which
            # is the printed row for "child 3 straggles".
            f = {0b000: 2, 0b001: 0, 0b010: 1, 0b100: 2}[straggler_mask]
            return A[f].copy()
        return decode_row(B, self.s, straggler_mask)


def execute(code: Code, local: list, G_parts: np.ndarray, masks) -> np.ndarray:
    """CR.Execute for one straggler pattern.  masks[g] is the straggler mask of
    sibling group g.  Leaves upload m = g_{D(L,i)}; a parent uploads
    m_(l,i) = a_f [m of its children] + g_{D(l,i)}; the master returns
    a_f [m_(1,1); ..; m_(1,n)].  Children with zero decode weight (stragglers
    and unused survivors) are never evaluated, nor are their sub-trees."""
    n, L = code.n, code.L

    def message(l: int, i: int) -> np.ndarray:
        v = flat_index(n, l, i)
        own = coded_gradient(local[v], G_parts)
        if l == L:
            return own
        return combine(l, i) + own

    def combine(l: int, i: int) -> np.ndarray:
        a = code.decode(l, int(masks[group_of_parent(n, l, i)]))
        total = np.zeros(G_parts.shape[1], dtype=np.float64)
        for j in range(1, n + 1):
            if a[j - 1] != 0.0:
                total += a[j - 1] * message(l + 1, n * (i - 1) + j)
        return total

    return combine(0, 1)


def execute_levels(code: Code, local: list, G_parts: np.ndarray, masks):
    """CR.Execute computed layer by layer for ALL nodes, as Algorithm 2 writes
    it (l = L-1 .. 1, then the master).  Returns (g, M) where M[l] is the
    (n**l, d) array of layer-l messages, l = 1..L.  Every group's mask must be
    decodable."""
    n, L = code.n, code.L
    E = encode_all(local, G_parts)
    M = {L: E[layer_offset(n, L): layer_offset(n, L) + n ** L].copy()}
    for l in range(L - 1, 0, -1):
        M[l] = np.zeros((n ** l, G_parts.shape[1]))
        for i in range(1, n ** l + 1):
            a = code.decode(l, int(masks[group_of_parent(n, l, i)]))
            kids = M[l + 1][n * (i - 1): n * i]
            M[l][i - 1] = a @ kids + E[flat_index(n, l, i)]
    a = code.decode(0, int(masks[0]))
    g = a @ M[1]
    return g, M


def used_nodes(code: Code, masks) -> list[int]:
    """Flat indices of the nodes whose local data enters the result for this
    straggler pattern (children with non-zero decode weight, recursively).
    Pinned by the node sets of the worked (3,2) example written out by hand
    and by the count sum_l (n-s)**l under exactly s stragglers per group."""
    n, L = code.n, code.L
    used = []

    def walk(l, i):
        a = code.decode(l, int(masks[group_of_parent(n, l, i)]))
        for j in range(1, n + 1):
            if a[j - 1] != 0.0:
                c = n * (i - 1) + j
                used.append(flat_index(n, l + 1, c))
                if l + 1 < L:
                    walk(l + 1, c)

    walk(0, 1)
    return sorted(used)


# --------------------------------------------------------------------------
# Plain definitions (Eq. g): what the whole method must reproduce
# --------------------------------------------------------------------------


def full_gradient(G_parts: np.ndarray) -> np.ndarray:
    """g = sum over all partitions of their gradients (Eq. g)."""
    return G_parts.astype(np.float64).sum(axis=0)


def partial_gradient_linreg(X: np.ndarray, y: np.ndarray, w: np.ndarray) -> np.ndarray:
    """Gradient of l(w) = 1/2 ||X w - y||^2 summed over the rows of one
    partition: X^T (X w - y), in fp64 from whatever precision the inputs have.
    Pinned by a central finite difference of the loss and by a 2 x 2 case
    worked by hand (gradient and loss as numbers)."""
    X = np.asarray(X, dtype=np.float64)
    return X.T @ (X @ np.asarray(w, dtype=np.float64) - np.asarray(y, dtype=np.float64))


def loss_linreg(X: np.ndarray, y: np.ndarray, w: np.ndarray) -> float:
    r = np.asarray(X, dtype=np.float64) @ np.asarray(w, dtype=np.float64) - np.asarray(y, dtype=np.float64)
    return 0.5 * float(r @ r)


def partial_gradient_logistic(X: np.ndarray, y: np.ndarray, w: np.ndarray) -> np.ndarray:
    """Gradient of the logistic loss sum_i [log(1 + exp(x_i.w)) - y_i x_i.w] over the rows of one
    partition (labels y in {0, 1}): X^T (sigmoid(X w) - y), the instance of Eq. (g) used in the
    paper's real-data experiment (Section V).  Pinned by a central finite difference of the loss and by
    the closed form at w = 0."""
    X = np.asarray(X, dtype=np.float64)
    z = X @ np.asarray(w, dtype=np.float64)
    return X.T @ (1.0 / (1.0 + np.exp(-z)) - np.asarray(y, dtype=np.float64))


def loss_logistic(X: np.ndarray, y: np.ndarray, w: np.ndarray) -> float:
    z = np.asarray(X, dtype=np.float64) @ np.asarray(w, dtype=np.float64)
    return float(np.sum(np.logaddexp(0.0, z) - np.asarray(y, dtype=np.float64) * z))


def normalized_error_rate(w: np.ndarray, w_star: np.ndarray) -> float:
    """||w - w*||^2 / ||w*||^2 (Eq. NER).  Pinned by a two-element case worked by hand."""
    w = w.astype(np.float64)
    w_star = w_star.astype(np.float64)
    return float(np.sum((w - w_star) ** 2) / np.sum(w_star ** 2))


# --------------------------------------------------------------------------
# Run-time model (Section III-C): shifted-exponential computation, single-port communication
# --------------------------------------------------------------------------


def expected_order_statistic(n: int, s: int, load_points: float, a: float, mu: float) -> float:
    """E[T_(n-s)] = (r d / mu) (H_n - H_s) + a r d for n i.i.d. shifted exponentials with shift
    a r d and rate mu / (r d) (Appendix D); load_points = r d."""
    H = lambda k: sum(1.0 / i for i in range(1, k + 1))
    return load_points / mu * (H(n) - H(s)) + a * load_points


def latency_trial(n: int, L: int, s: int, compute_time, t_c: float):
    """One run of CR.Execute on the clock.  A leaf's message is ready when its computation ends.  A parent
    listens to one child at a time (single-port model, a message takes t_c), serving children in the
    order in which their messages become ready (ties: lower index), and stops after n-s messages; its own
    message is ready when it has those and its own computation has ended.  Returns (masks, T): per
    sibling group the bit mask of the s children not waited for, and the time at which the master has
    its n-s messages.  Pinned by hand-worked cases, by the order-statistic mean of Appendix D (t_c = 0)
    and by elementary bounds."""
    ready = {}
    masks = [0] * num_groups(n, L)

    def serve(l, i):
        """Time at which parent (l, i) holds n-s messages; records its group's mask."""
        kids = []
        for j in range(1, n + 1):
            c = n * (i - 1) + j
            kids.append((message_ready(l + 1, c), j - 1))
        kids.sort()                       # by ready time, then by index
        port_free = 0.0
        got = 0.0
        for rank, (t_ready, j) in enumerate(kids):
            if rank < n - s:
                port_free = max(t_ready, port_free) + t_c
                got = port_free
            else:
                masks[group_of_parent(n, l, i)] |= 1 << j
        return got

    def message_ready(l, i):
        if (l, i) not in ready:
            own = float(compute_time[flat_index(n, l, i)])
            ready[(l, i)] = own if l == L else max(serve(l, i), own)
        return ready[(l, i)]

    total = serve(0, 1)
    return masks, total


# --------------------------------------------------------------------------
# Integer-exact mode
# --------------------------------------------------------------------------


def integer_scale(code: Code) -> int:
    """Smallest power-of-two sigma for which sigma * B is integer at every level
    (2 for the printed code, 1 for 0/1 repetition).  With S = sigma**L every
    coefficient S * c of every node is an integer, so the whole tree can be run
    on S * (true values) in integers and divided by S at the root."""
    sigma = 1
    while any(np.any(np.abs(B * sigma - np.round(B * sigma)) > 0) for B in code.B_levels):
        sigma *= 2
        if sigma > 1 << 20:
            raise ValueError("B is not dyadic: no integer form")
    return sigma


def execute_integer(code: Code, local: list, G_parts_int: np.ndarray, masks) -> np.ndarray:
    """Integer-exact CR.Execute with Python/NumPy int64 arithmetic: run the
    recursion of `execute` on S * c (integers) and divide exactly by
    S = sigma**L at the root."""
    n, L = code.n, code.L
    S = integer_scale(code) ** L

    def as_int(x: float) -> int:
        r = round(x)
        assert r == x, "coefficient is not an integer"
        return int(r)

    def message(l, i):
        v = flat_index(n, l, i)
        own = np.zeros(G_parts_int.shape[1], dtype=np.int64)
        for p, c in local[v]:
            own += as_int(c * S) * G_parts_int[p].astype(np.int64)
        if l == L:
            return own
        return combine(l, i) + own

    def combine(l, i):
        a = code.decode(l, int(masks[group_of_parent(n, l, i)]))
        total = np.zeros(G_parts_int.shape[1], dtype=np.int64)
        for j in range(1, n + 1):
            if a[j - 1] != 0.0:
                total += as_int(a[j - 1]) * message(l + 1, n * (i - 1) + j)
        return total

    scaled = combine(0, 1)
    assert np.all(scaled % S == 0), "scaled result is not divisible by the scale"
    return scaled // S
