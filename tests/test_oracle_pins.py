"""Pins for the CPU oracle: every check compares it with something other than itself --
hand-derived values, brute force written independently in numpy/Python, algebraic identities
the paper states, closed forms and library routines."""
import itertools

import numpy as np
import pytest

import oracle


def _offsets(w):
    return np.concatenate([[0], np.cumsum(w)]).astype(int)


def _rand_ints(rng, shape, lo=-3, hi=3):
    return rng.integers(lo, hi + 1, size=shape).astype(np.float64)


# ---- P7: hand-derived examples (tests/golden/hand_examples.json) ------------------------------

@pytest.mark.parametrize("key", ["typed_q2", "typed_q3"])
def test_hand_examples_typed(golden, key):
    g = golden[key]
    W = np.array(g["W"], dtype=np.float64)
    x = np.array(g["x"], dtype=np.float64)
    q = len(x)
    ones = [1] * q
    for t, want in enumerate(g["y_by_type"]):
        for form in ("rows", "alg1"):
            got = oracle.proj(x[None, :], [t], W, ones, ones, form=form)
            assert got.tolist() == [list(map(float, want))], (key, t, form)
    dense = oracle.proj(x[None, :], [0], W, ones, ones, keep=oracle.support(q, "dense"))
    assert dense.tolist() == [list(map(float, g["dense"]))]


def test_hand_example_square(golden):
    g = golden["square_q2"]
    A, B, C = (np.array(g[k], dtype=np.float64) for k in "ABC")
    one = [1, 1]
    AB = oracle.square(A, B, one, one, one)
    BC = oracle.square(B, C, one, one, one)
    assert AB.tolist() == g["A_star_B"]
    assert BC.tolist() == g["B_star_C"]
    assert oracle.square(AB, C, one, one, one).tolist() == g["ABC"]
    assert oracle.square(A, BC, one, one, one).tolist() == g["ABC"]


# ---- P1: the six-product rule, term by term ---------------------------------------------------

def test_q2_six_products_term_by_term():
    """One-hot block probes: X group k and W block (k', j) non-zero. The output block j of a
    type-t row is non-zero iff k == k' and k in {t, j}; for q=2 exactly A Wa, A Wu, U Wd,
    V Wa, D Wv, D Wd survive and U Wv, V Wu never appear (Eq. six-product)."""
    q, s, r = 2, [2, 3], [3, 2]
    so, ro = _offsets(s), _offsets(r)
    rng = np.random.default_rng(1)
    survivors = set()
    for t, k, kp, j in itertools.product(range(q), repeat=4):
        X = np.zeros((1, sum(s)))
        W = np.zeros((sum(s), sum(r)))
        X[0, so[k]:so[k + 1]] = rng.integers(1, 4, size=s[k])
        W[so[kp]:so[kp + 1], ro[j]:ro[j + 1]] = rng.integers(1, 4, size=(s[kp], r[j]))
        Y = oracle.proj(X, [t], W, s, r)
        nz = bool(np.any(Y != 0))
        assert nz == (k == kp and k in (t, j)), (t, k, kp, j)
        if nz:
            assert np.array_equal(Y, X @ W)
            outside = np.ones(sum(r), bool)
            outside[ro[j]:ro[j + 1]] = False
            assert not np.any(Y[0, outside])
            survivors.add((t, k, j))
    # (type, activation group, output group): A=(0,0) U=(0,1) V=(1,0) D=(1,1)
    assert survivors == {(0, 0, 0), (0, 0, 1), (0, 1, 1), (1, 0, 0), (1, 1, 0), (1, 1, 1)}
    assert (0, 1, 0) not in survivors and (1, 0, 1) not in survivors  # U Wv and V Wu


@pytest.mark.parametrize("q", [3, 4, 5])
def test_support_probe_general_q(q):
    keep = oracle.support(q)
    for i, j, k in itertools.product(range(q), repeat=3):
        assert bool(keep[i, j, k]) == (k in (i, j))


def test_large_algebra_rows_against_the_two_stage_form():
    """Fixed-block regime (q in the hundreds, blocks off the tile grid): the per-row equation equals the
    two-stage form of Section "Kernels" -- the block-diagonal map x_j W_jj for every row, then x_i W_ij
    for the off-diagonal groups of a type-i row -- written here with numpy slices; counts follow Eq. q-rank."""
    q, s, r, M = 72, 3, 5, 40
    rng = np.random.default_rng(72)
    X = _rand_ints(rng, (M, q * s))
    W = _rand_ints(rng, (q * s, q * r))
    types = rng.integers(0, q, size=M)
    Y = np.zeros((M, q * r))
    for j in range(q):                                   # stage 1: diagonal blocks, all rows
        Y[:, j * r:(j + 1) * r] = X[:, j * s:(j + 1) * s] @ W[j * s:(j + 1) * s, j * r:(j + 1) * r]
    for b in range(M):                                   # stage 2: the row panel of the row's own type
        i = types[b]
        panel = X[b, i * s:(i + 1) * s] @ W[i * s:(i + 1) * s, :]
        panel[i * r:(i + 1) * r] = 0                     # B(i,i) = {i}: counted once, in stage 1
        Y[b] += panel
    assert np.array_equal(oracle.proj(X, types, W, [s] * q, [r] * q), Y)
    keep = oracle.support(q)
    assert oracle.gemm_count(keep) == 2 * q * q - q
    rows = np.bincount(types, minlength=q)
    assert oracle.macs(keep, [s] * q, [r] * q, rows) == M * (2 * q - 1) * s * r


# ---- P2: counts and MAC formulas -------------------------------------------------------------

def test_gemm_counts(golden):
    for q, n in golden["gemm_counts"]["qq"].items():
        q = int(q)
        keep = oracle.support(q)
        assert oracle.gemm_count(keep) == n == 2 * q * q - q
        assert all(int(keep[i].sum()) == 2 * q - 1 for i in range(q))
        assert oracle.gemm_count(oracle.support(q, "dense")) == q ** 3
    for q, n in golden["gemm_counts"]["q2pow"].items():
        assert oracle.gemm_count(oracle.support(int(q), "q2pow")) == n


def test_mac_formulas():
    rng = np.random.default_rng(2)
    for q in (2, 3, 4, 7):
        s = rng.integers(1, 9, size=q)
        r = rng.integers(1, 9, size=q)
        rows = rng.integers(0, 50, size=q)
        keep = oracle.support(q)
        d_diag = int((s * r).sum())
        N = int(r.sum())
        want = int(rows.sum()) * d_diag + int(sum(rows[i] * s[i] * (N - r[i]) for i in range(q)))
        assert oracle.macs(keep, s, r, rows) == want  # Eq. rectangular-batch-cost
    for q in (2, 4, 8, 16):  # equal groups: rho_q = (2q-1)/q^2
        s, r, rows = [6] * q, [10] * q, [3] * q
        M, K, N = 3 * q, 6 * q, 10 * q
        assert oracle.macs(oracle.support(q), s, r, rows) * q * q == (2 * q - 1) * M * K * N
    # tensor power: ratio (3/4)^L with equal groups and equally frequent types
    for L in (1, 2, 3):
        q = 2 ** L
        m = oracle.macs(oracle.support(q, "q2pow"), [4] * q, [4] * q, [5] * q)
        assert m * 4 ** L == 3 ** L * (5 * q) * (4 * q) * (4 * q)


# ---- P3: dense minus the removed products (brute force, independent numpy) --------------------

@pytest.mark.parametrize("q", [2, 3, 4])
def test_dense_minus_removed(q):
    rng = np.random.default_rng(10 + q)
    s = rng.integers(1, 4, size=q)
    r = rng.integers(1, 4, size=q)
    so, ro = _offsets(s), _offsets(r)
    M = 8
    X = _rand_ints(rng, (M, s.sum()))
    W = _rand_ints(rng, (s.sum(), r.sum()))
    types = rng.integers(0, q, size=M)
    want = X @ W
    for b in range(M):
        for j in range(q):
            for k in range(q):
                if k not in (types[b], j):
                    want[b, ro[j]:ro[j + 1]] -= X[b, so[k]:so[k + 1]] @ W[so[k]:so[k + 1], ro[j]:ro[j + 1]]
    for form in ("rows", "alg1"):
        assert np.array_equal(oracle.proj(X, types, W, s, r, form=form), want)


@pytest.mark.parametrize("q", [2, 3, 4])
def test_single_entries_against_dense_minus_removed(q):
    """proj_entries sums one output at a time; pinned by the same independent numpy statement
    (dense product minus the removed block products), with a bias, on every (row, column)."""
    rng = np.random.default_rng(40 + q)
    s = rng.integers(1, 4, size=q)
    r = rng.integers(1, 4, size=q)
    so, ro = _offsets(s), _offsets(r)
    M = 7
    X = _rand_ints(rng, (M, s.sum()))
    W = _rand_ints(rng, (s.sum(), r.sum()))
    bias = _rand_ints(rng, (r.sum(),))
    types = rng.integers(0, q, size=M)
    want = X @ W + bias
    for b in range(M):
        for j in range(q):
            for k in range(q):
                if k not in (types[b], j):
                    want[b, ro[j]:ro[j + 1]] -= X[b, so[k]:so[k + 1]] @ W[so[k]:so[k + 1], ro[j]:ro[j + 1]]
    rows, cols = np.meshgrid(np.arange(M), np.arange(r.sum()), indexing="ij")
    got = oracle.proj_entries(X, types, W, s, r, rows.ravel(), cols.ravel(), bias=bias)
    assert np.array_equal(got.reshape(M, -1), want)
    with pytest.raises(oracle.OracleError):
        oracle.proj_entries(X, types, W, s, r, [M], [0])


def test_ffn_entries_and_gelu_array():
    """ffn_entries against an independent numpy composition (q = 2, dense minus the removed product)."""
    import math
    rng = np.random.default_rng(61)
    q, dw, fw = 2, [3, 2], [4, 5]
    M = 9
    X = rng.standard_normal((M, 5))
    Wu = rng.standard_normal((5, 9))
    Wd = rng.standard_normal((9, 5))
    bu, bd = rng.standard_normal(9), rng.standard_normal(5)
    types = rng.integers(0, q, size=M)
    z = np.linspace(-5, 5, 23)
    np.testing.assert_allclose(oracle.gelu_array(z), [0.5 * v * math.erfc(-v / math.sqrt(2)) for v in z], atol=1e-14)

    def star2(Xm, Wm, s, r, bias):
        so, ro = _offsets(s), _offsets(r)
        out = Xm @ Wm + bias
        for b, t in enumerate(types):
            o = 1 - t
            out[b, ro[t]:ro[t + 1]] -= Xm[b, so[o]:so[o + 1]] @ Wm[so[o]:so[o + 1], ro[t]:ro[t + 1]]
        return out
    Hn = np.vectorize(lambda v: 0.5 * v * (1 + math.erf(v / math.sqrt(2))))(star2(X, Wu, dw, fw, bu))
    want = star2(Hn, Wd, fw, dw, bd)
    rows = np.array([0, 8, 3, 3, 5, 8])
    cols = np.array([0, 4, 2, 3, 1, 0])
    got = oracle.ffn_entries(X, types, Wu, Wd, dw, fw, rows, cols, b_up=bu, b_down=bd)
    np.testing.assert_allclose(got, want[rows, cols], rtol=1e-12, atol=1e-12)


def test_pure_python_scalar_loops():
    """Scalar-level restatement of Eqs. typed-diag/off with explicit Python loops."""
    rng = np.random.default_rng(5)
    q, s, r = 3, [2, 1, 3], [1, 2, 2]
    so, ro = _offsets(s), _offsets(r)
    X = _rand_ints(rng, (6, 6))
    W = _rand_ints(rng, (6, 5))
    types = [0, 1, 2, 2, 1, 0]
    want = np.zeros((6, 5))
    for b, i in enumerate(types):
        for j in range(q):
            for n in range(ro[j], ro[j + 1]):
                acc = 0.0
                for c in range(so[i], so[i + 1]):        # x_i W_ij
                    acc += X[b, c] * W[c, n]
                if j != i:
                    for c in range(so[j], so[j + 1]):    # + x_j W_jj
                        acc += X[b, c] * W[c, n]
                want[b, n] = acc
    assert np.array_equal(oracle.proj(X, types, W, s, r), want)


# ---- P4, P5, P8: associativity, unit, edge ideal on integer block arrays ---------------------

def _np_square_star(A, B, q, b):
    """Independent numpy statement of (d,n)*(d',n') = (dd', dn' + nd') (Appendix A)."""
    C = np.zeros_like(A)
    blk = lambda Z, i, j: Z[i * b:(i + 1) * b, j * b:(j + 1) * b]
    for i in range(q):
        for j in range(q):
            if i == j:
                blk(C, i, i)[:] = blk(A, i, i) @ blk(B, i, i)
            else:
                blk(C, i, j)[:] = blk(A, i, i) @ blk(B, i, j) + blk(A, i, j) @ blk(B, j, j)
    return C


@pytest.mark.parametrize("q,b", [(2, 1), (2, 3), (3, 2), (4, 2), (4, 3)])
def test_associativity_unit_ideal(q, b):
    rng = np.random.default_rng(100 * q + b)
    n = q * b
    w = [b] * q
    X, Y, Z = (_rand_ints(rng, (n, n), -2, 2) for _ in range(3))
    star = lambda P, Q: oracle.square(P, Q, w, w, w)
    assert np.array_equal(star(X, Y), _np_square_star(X, Y, q, b))
    assert np.array_equal(star(star(X, Y), Z), star(X, star(Y, Z)))
    E = np.eye(n)
    assert np.array_equal(star(E, X), X) and np.array_equal(star(X, E), X)
    # two arrays with zero diagonal blocks multiply to zero (J^2 = 0)
    mask = np.kron(1 - np.eye(q), np.ones((b, b)))
    assert not np.any(star(X * mask, Y * mask))
    # the rule is not ordinary matrix multiplication
    assert not np.array_equal(star(X, Y), X @ Y)


def test_associativity_rectangular_blocks():
    rng = np.random.default_rng(77)
    a, c, d, e = [2, 1, 3], [1, 2, 2], [3, 1, 1], [2, 2, 1]
    X = _rand_ints(rng, (sum(a), sum(c)))
    Y = _rand_ints(rng, (sum(c), sum(d)))
    Z = _rand_ints(rng, (sum(d), sum(e)))
    left = oracle.square(oracle.square(X, Y, a, c, d), Z, a, d, e)
    right = oracle.square(X, oracle.square(Y, Z, c, d, e), a, c, e)
    assert np.array_equal(left, right)


# ---- P6: typed rows <-> square display, and the composition law ------------------------------

def test_typed_rows_match_square_display():
    """Row block i of the square product is the typed projection of rows of type i."""
    rng = np.random.default_rng(8)
    q, a, c, d = 3, [2, 3, 1], [2, 1, 2], [1, 3, 2]
    A = _rand_ints(rng, (sum(a), sum(c)))
    B = _rand_ints(rng, (sum(c), sum(d)))
    types = np.repeat(np.arange(q), a)
    assert np.array_equal(oracle.proj(A, types, B, c, d), oracle.square(A, B, a, c, d))


def test_composition_law():
    """Phi_{W2}(Phi_{W1}(X)) = Phi_{W1 * W2}(X) for row-typed X (Eq. association-intro)."""
    rng = np.random.default_rng(9)
    q, s, m, r = 3, [2, 1, 2], [1, 3, 2], [2, 2, 1]
    M = 11
    X = _rand_ints(rng, (M, sum(s)))
    W1 = _rand_ints(rng, (sum(s), sum(m)))
    W2 = _rand_ints(rng, (sum(m), sum(r)))
    types = rng.integers(0, q, size=M)
    lhs = oracle.proj(oracle.proj(X, types, W1, s, m), types, W2, m, r)
    rhs = oracle.proj(X, types, oracle.square(W1, W2, s, m, r), s, r)
    assert np.array_equal(lhs, rhs)


# ---- P9: reductions to library routines and closed forms -------------------------------------

def test_dense_table_and_q1_are_matmul():
    rng = np.random.default_rng(3)
    X = rng.standard_normal((17, 12))
    W = rng.standard_normal((12, 10))
    types = rng.integers(0, 3, size=17)
    Y = oracle.proj(X, types, W, [3, 4, 5], [2, 5, 3], keep=oracle.support(3, "dense"))
    np.testing.assert_allclose(Y, X @ W, rtol=1e-13, atol=1e-13)
    Y1 = oracle.proj(X, np.zeros(17, int), W, [12], [10])
    np.testing.assert_allclose(Y1, X @ W, rtol=1e-13, atol=1e-13)
    bias = rng.standard_normal(10)
    Yb = oracle.proj(X, np.zeros(17, int), W, [12], [10], bias=bias)
    np.testing.assert_allclose(Yb, X @ W + bias, rtol=1e-13, atol=1e-13)


def test_rows_vs_alg1_float():
    rng = np.random.default_rng(4)
    q, s, r = 4, [3, 5, 2, 4], [4, 1, 6, 2]
    X = rng.standard_normal((23, sum(s)))
    W = rng.standard_normal((sum(s), sum(r)))
    types = rng.integers(0, q, size=23)
    np.testing.assert_allclose(oracle.proj(X, types, W, s, r, form="rows"),
                               oracle.proj(X, types, W, s, r, form="alg1"), rtol=1e-12, atol=1e-12)


def test_gelu_closed_form(golden):
    for z, want in golden["gelu"]["points"]:
        assert abs(oracle.gelu(z) - want) < 5e-10
    import math
    for z in np.linspace(-6, 6, 41):
        assert abs(oracle.gelu(z) - 0.5 * z * math.erfc(-z / math.sqrt(2))) < 1e-14


def test_ffn_composes_projections():
    rng = np.random.default_rng(6)
    q, dw, fw = 2, [3, 2], [4, 5]
    M = 9
    X = rng.standard_normal((M, 5))
    Wu = rng.standard_normal((5, 9))
    Wd = rng.standard_normal((9, 5))
    bu, bd = rng.standard_normal(9), rng.standard_normal(5)
    types = rng.integers(0, q, size=M)
    Y, H = oracle.ffn(X, types, Wu, Wd, dw, fw, b_up=bu, b_down=bd, return_hidden=True)
    # independent numpy composition using the dense-minus-removed statement for q=2
    def star2(Xm, Wm, s, r, bias):
        so, ro = _offsets(s), _offsets(r)
        out = Xm @ Wm + bias
        for b, t in enumerate(types):
            o = 1 - t  # the removed product for a type-t row is x_o W_{o,t}
            out[b, ro[t]:ro[t + 1]] -= Xm[b, so[o]:so[o + 1]] @ Wm[so[o]:so[o + 1], ro[t]:ro[t + 1]]
        return out
    import math
    Hn = star2(X, Wu, dw, fw, bu)
    Hn = np.vectorize(lambda z: 0.5 * z * (1 + math.erf(z / math.sqrt(2))))(Hn)
    np.testing.assert_allclose(H, Hn, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(Y, star2(Hn, Wd, fw, dw, bd), rtol=1e-12, atol=1e-12)


def test_silu_closed_form(golden):
    import math
    for z, want in golden["silu"]["points"]:
        assert abs(oracle.silu(z) - want) < 1e-12
    for z in np.linspace(-8, 8, 33):
        assert abs(oracle.silu(z) - z * 0.5 * (1.0 + math.tanh(0.5 * z))) < 1e-13      # z * sigmoid(z), another form


def test_gated_ffn_composes_three_projections():
    """SwiGLU FFN against an independent numpy composition (q = 2: dense minus the removed product;
    q = 4 tensor-square law: per-row sums written from the bit rule)."""
    rng = np.random.default_rng(7)
    q, dw, fw = 2, [3, 2], [4, 5]
    M = 9
    X = rng.standard_normal((M, 5))
    Wg, Wu = rng.standard_normal((5, 9)), rng.standard_normal((5, 9))
    Wd = rng.standard_normal((9, 5))
    types = rng.integers(0, q, size=M)

    def star2(Xm, Wm, s, r):
        so, ro = _offsets(s), _offsets(r)
        out = Xm @ Wm
        for b, t in enumerate(types):
            o = 1 - t
            out[b, ro[t]:ro[t + 1]] -= Xm[b, so[o]:so[o + 1]] @ Wm[so[o]:so[o + 1], ro[t]:ro[t + 1]]
        return out
    G, U = star2(X, Wg, dw, fw), star2(X, Wu, dw, fw)
    Hn = G / (1.0 + np.exp(-G)) * U
    Y, Hh = oracle.ffn_swiglu(X, types, Wg, Wu, Wd, dw, fw, return_hidden=True)
    np.testing.assert_allclose(Hh, Hn, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(Y, star2(Hn, Wd, fw, dw), rtol=1e-12, atol=1e-12)
    # tensor-square law, q = 4: group beta enters output group delta of a type-alpha row iff every
    # bit of beta equals that bit of alpha or of delta
    q, dw, fw = 4, [2, 1, 2, 1], [1, 2, 1, 2]
    X = rng.standard_normal((6, 6))
    Wg, Wu, Wd = rng.standard_normal((6, 6)), rng.standard_normal((6, 6)), rng.standard_normal((6, 6))
    types = np.array([0, 1, 2, 3, 2, 1])
    keep = oracle.support(4, "q2pow")

    def star_pow(Xm, Wm, s, r):
        so, ro = _offsets(s), _offsets(r)
        out = np.zeros((Xm.shape[0], ro[-1]))
        for b, al in enumerate(types):
            for de in range(4):
                for be in range(4):
                    if all(((be >> k) & 1) in (((al >> k) & 1), ((de >> k) & 1)) for k in range(2)):
                        out[b, ro[de]:ro[de + 1]] += Xm[b, so[be]:so[be + 1]] @ Wm[so[be]:so[be + 1], ro[de]:ro[de + 1]]
        return out
    G, U = star_pow(X, Wg, dw, fw), star_pow(X, Wu, dw, fw)
    Hn = G / (1.0 + np.exp(-G)) * U
    np.testing.assert_allclose(oracle.ffn_swiglu(X, types, Wg, Wu, Wd, dw, fw, keep=keep), star_pow(Hn, Wd, fw, dw),
                               rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("q", [2, 3, 4])
def test_vjp_against_the_displayed_per_type_equations(q):
    """Eqs. vjp-xi ... vjp-wjj, typed out per token of type i in numpy (integers: exact)."""
    rng = np.random.default_rng(70 + q)
    s = rng.integers(1, 4, size=q)
    r = rng.integers(1, 4, size=q)
    so, ro = _offsets(s), _offsets(r)
    M = 11
    X = _rand_ints(rng, (M, s.sum()))
    W = _rand_ints(rng, (s.sum(), r.sum()))
    G = _rand_ints(rng, (M, r.sum()))
    types = rng.integers(0, q, size=M)
    dX, dW = np.zeros_like(X), np.zeros_like(W)
    blk = lambda A, a, b, ao, bo: A[ao[a]:ao[a + 1], bo[b]:bo[b + 1]]
    for b in range(M):
        i = types[b]
        x = lambda k: X[b, so[k]:so[k + 1]]
        g = lambda j: G[b, ro[j]:ro[j + 1]]
        dX[b, so[i]:so[i + 1]] += g(i) @ blk(W, i, i, so, ro).T + sum(g(j) @ blk(W, i, j, so, ro).T for j in range(q) if j != i)
        dW[so[i]:so[i + 1], ro[i]:ro[i + 1]] += np.outer(x(i), g(i))
        for j in range(q):
            if j == i:
                continue
            dX[b, so[j]:so[j + 1]] += g(j) @ blk(W, j, j, so, ro).T
            dW[so[i]:so[i + 1], ro[j]:ro[j + 1]] += np.outer(x(i), g(j))
            dW[so[j]:so[j + 1], ro[j]:ro[j + 1]] += np.outer(x(j), g(j))
    assert np.array_equal(oracle.proj_vjp_x(G, types, W, s, r), dX)
    assert np.array_equal(oracle.proj_vjp_w(X, G, types, s, r), dW)


@pytest.mark.parametrize("law,q", [("qq", 3), ("q2pow", 4), ("dense", 2)])
def test_vjp_adjoint_identities(law, q):
    """The projection is bilinear in (X, W): <X * W, G> = <X, dX(G)> = <W, dW(X, G)>, exactly on integers,
    for every support set; a missing type leaves its private blocks of dW at zero."""
    rng = np.random.default_rng(80 + q)
    s = rng.integers(1, 4, size=q)
    r = rng.integers(1, 4, size=q)
    so, ro = _offsets(s), _offsets(r)
    keep = oracle.support(q, law)
    M = 13
    X = _rand_ints(rng, (M, s.sum()))
    W = _rand_ints(rng, (s.sum(), r.sum()))
    G = _rand_ints(rng, (M, r.sum()))
    types = rng.integers(0, q - 1, size=M) if q > 1 else np.zeros(M, int)     # the last type is absent
    Y = oracle.proj(X, types, W, s, r, keep=keep)
    dX = oracle.proj_vjp_x(G, types, W, s, r, keep=keep)
    dW = oracle.proj_vjp_w(X, G, types, s, r, keep=keep)
    assert np.sum(Y * G) == np.sum(X * dX) == np.sum(W * dW)
    if law == "qq":   # W_{q-1, j} (j != q-1) is used by rows of type q-1 only
        assert not dW[so[q - 1]:so[q], :ro[q - 1]].any()
    # second probe with one-hot gradients pins single entries, not only the sum
    for (b, n) in [(0, 0), (M - 1, int(r.sum()) - 1), (5, int(ro[1]))]:
        E = np.zeros_like(G)
        E[b, n] = 1.0
        assert np.array_equal(oracle.proj_vjp_x(E, types, W, s, r, keep=keep)[b],
                              np.array([(oracle.proj(np.eye(1, int(s.sum()), c), [types[b]], W, s, r, keep=keep))[0, n]
                                        for c in range(int(s.sum()))]))


def test_vjp_dense_table_is_the_matmul_transpose_pair():
    """With every block kept the projection is X @ W, so its gradient maps are G @ W^T and X^T @ G; a one-hot
    weight perturbation pins single entries of dW for the Q_q law (the map is linear in W)."""
    rng = np.random.default_rng(91)
    s, r = np.array([2, 1, 3]), np.array([1, 2, 2])
    M = 9
    X = _rand_ints(rng, (M, s.sum()))
    W = _rand_ints(rng, (s.sum(), r.sum()))
    G = _rand_ints(rng, (M, r.sum()))
    types = rng.integers(0, 3, size=M)
    keep = oracle.support(3, "dense")
    assert np.array_equal(oracle.proj_vjp_x(G, types, W, s, r, keep=keep), G @ W.T)
    assert np.array_equal(oracle.proj_vjp_w(X, G, types, s, r, keep=keep), X.T @ G)
    dW = oracle.proj_vjp_w(X, G, types, s, r)
    for (k, n) in [(0, 0), (int(s.sum()) - 1, int(r.sum()) - 1), (2, 1), (3, 0)]:
        E = np.zeros_like(W)
        E[k, n] = 1.0
        assert dW[k, n] == np.sum(oracle.proj(X, types, E, s, r) * G)


def test_bad_type_rejected():
    with pytest.raises(oracle.OracleError):
        oracle.proj(np.zeros((2, 2)), [0, 2], np.zeros((2, 2)), [1, 1], [1, 1])
    with pytest.raises(oracle.OracleError):
        oracle.proj(np.zeros((2, 2)), [0, -1], np.zeros((2, 2)), [1, 1], [1, 1], form="alg1")


def test_empty_and_missing_types():
    Y = oracle.proj(np.zeros((0, 4)), np.zeros(0, int), np.ones((4, 6)), [2, 2], [3, 3])
    assert Y.shape == (0, 6)
    X = np.ones((3, 4))
    Y = oracle.proj(X, [1, 1, 1], np.ones((4, 6)), [2, 2], [3, 3])  # no type-0 rows at all
    assert np.array_equal(Y, np.tile([4, 4, 4, 2, 2, 2], (3, 1)).astype(float))


def test_tensor_power_support_is_kronecker_product_of_q2():
    """B(alpha, delta) of Q_2^{(x)L} factorises bit by bit into the q=2 rule (appendix on the
    tensor-square candidate): keep_L[a,d,b] = prod_bits keep_2[a_bit, d_bit, b_bit]."""
    k2 = oracle.support(2)
    for L in (1, 2, 3):
        q = 2 ** L
        kL = oracle.support(q, "q2pow")
        for a, d, b in itertools.product(range(q), repeat=3):
            want = 1
            for bit in range(L):
                want *= int(k2[(a >> bit) & 1, (d >> bit) & 1, (b >> bit) & 1])
            assert int(kL[a, d, b]) == want
        # per-type product count 3^L, total 6^L; strictly between the direct law and dense for L >= 2
        assert all(int(kL[a].sum()) == 3 ** L for a in range(q))
    assert oracle.gemm_count(oracle.support(4, "q2pow")) == 36 > oracle.gemm_count(oracle.support(4)) == 28
