"""Pins for the CPU oracle: every check compares the C loops against something
other than themselves - Definition 3.1 materialised literally, closed forms,
finite differences, textbook values, and the projection invariant."""
import math
import os

import numpy as np
import pytest

from oracle import monarch_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(rng, *shape):
    return rng.standard_normal(shape)


def _read_table(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append([float(v) for v in line.split()])
    return np.array(rows)


# ------------------------------------------------------------------ permutation

def test_perm_matches_definition_listing():
    # Definition 3.1 lists the order of the permuted vector.
    listed = _read_table("perm_m3.txt")[0].astype(int) - 1
    P = O.perm_matrix(3)
    x = np.arange(9, dtype=np.float64)
    assert np.array_equal(P @ x, x[listed])


@pytest.mark.parametrize("m", [2, 3, 4, 8])
def test_perm_is_symmetric_involution(m):
    # Section 3.1: "Note that P = P^T"; hence P P = I.
    P = O.perm_matrix(m)
    assert np.array_equal(P, P.T)
    assert np.array_equal(P @ P, np.eye(m * m))
    x = np.arange(m * m, dtype=np.float64)
    assert np.array_equal(P @ x, x.reshape(m, m).T.reshape(-1))


@pytest.mark.parametrize("m", [2, 3, 4])
def test_PtLP_is_grid_of_diagonal_blocks(m):
    # Section 3.1: L' = P^T L P consists of m x m blocks, each diagonal.
    rng = np.random.default_rng(1)
    L = _rand(rng, m, m, m)
    P = O.perm_matrix(m)
    Lp = P.T @ O.blockdiag(L) @ P
    for a in range(m):
        for b in range(m):
            D = Lp[a * m:(a + 1) * m, b * m:(b + 1) * m]
            assert np.array_equal(D, np.diag(np.diag(D)))
            assert np.allclose(np.diag(D), L[:, a, b], rtol=0, atol=0)


# ------------------------------------------------------------------ forward

@pytest.mark.parametrize("m", [2, 3, 4, 8])
def test_three_routes_agree(m):
    # Definition 3.1 (explicit P, blockdiag), Eq. (2), and steps 1-3.
    rng = np.random.default_rng(10 + m)
    n = m * m
    L, R = _rand(rng, m, m, m), _rand(rng, m, m, m)
    x = _rand(rng, 5, n)
    M_def = O.dense_from_definition(L, R)
    M_eq2 = O.dense(L, R)
    assert np.allclose(M_def, M_eq2, rtol=1e-13, atol=1e-13)
    y = O.fwd(x, L, R)
    assert np.allclose(y, x @ M_def.T, rtol=1e-12, atol=1e-12)


def test_eq2_entry_formula_explicit():
    # M[(l)m+j, (k)m+i] = L[j,l,k] R[k,j,i], spelled with numpy's einsum as a
    # second statement of Eq. (2).
    rng = np.random.default_rng(3)
    m = 4
    L, R = _rand(rng, m, m, m), _rand(rng, m, m, m)
    M4 = np.einsum("jlk,kji->ljki", L, R)
    assert np.allclose(O.dense(L, R), M4.reshape(m * m, m * m), rtol=0, atol=1e-15)
    assert np.allclose(O.dense_from_definition(L, R), M4.reshape(m * m, m * m), atol=1e-13)


@pytest.mark.parametrize("m", [3, 4])
def test_stage_isolation(m):
    rng = np.random.default_rng(4)
    n = m * m
    W = _rand(rng, m, m, m)
    I = np.stack([np.eye(m)] * m)
    x = _rand(rng, 3, n)
    # L = I: M = P P^T R = blockdiag(R)
    y = O.fwd(x, I, W)
    assert np.allclose(y, x @ O.blockdiag(W).T, atol=1e-13)
    # R = I: M = P L P^T, entries delta_{ji} L[j,l,k]
    y = O.fwd(x, W, I)
    P = O.perm_matrix(m)
    assert np.allclose(y, x @ (P @ O.blockdiag(W) @ P.T).T, atol=1e-13)
    u_expected = x.reshape(3, m, m)                           # u = x when R = I
    _, u = O.fwd(x, W, I, return_u=True)
    assert np.array_equal(u, u_expected)


@pytest.mark.parametrize("m", [2, 3, 5])
def test_kronecker_closed_form(m):
    # Identical blocks: L_j = A, R_k = B  =>  M = A (x) B  (from Eq. (2)).
    rng = np.random.default_rng(5)
    A, B = _rand(rng, m, m), _rand(rng, m, m)
    L = np.stack([A] * m)
    R = np.stack([B] * m)
    x = _rand(rng, 4, m * m)
    assert np.allclose(O.dense(L, R), np.kron(A, B), atol=1e-14)
    assert np.allclose(O.fwd(x, L, R), x @ np.kron(A, B).T, atol=1e-12)


def _sylvester(m):
    H = np.array([[1.0]])
    while H.shape[0] < m:
        H = np.block([[H, H], [H, -H]])
    return H


def test_hadamard_h4_golden():
    H4 = _read_table("hadamard_h4.txt")
    H2 = _sylvester(2)
    L = np.stack([H2] * 2)
    R = np.stack([H2] * 2)
    assert np.array_equal(O.dense(L, R), H4)
    assert np.array_equal(O.dense_from_definition(L, R), H4)


@pytest.mark.parametrize("m", [2, 4, 8, 16])
def test_hadamard_transform_exact(m):
    # All blocks H_m  =>  M = H_n in natural (Sylvester) order:
    # y[a] = sum_b (-1)^{popcount(a & b)} x[b].  Small integers: exact.
    n = m * m
    rng = np.random.default_rng(6)
    x = rng.integers(-3, 4, size=(3, n)).astype(np.float64)
    Hm = _sylvester(m)
    y = O.fwd(x, np.stack([Hm] * m), np.stack([Hm] * m))
    a = np.arange(n)
    sign = np.array([[(-1) ** bin(p & q).count("1") for q in a] for p in a], dtype=np.float64)
    assert np.array_equal(y, x @ sign.T)


def test_forward_edge_token_counts():
    rng = np.random.default_rng(7)
    m = 4
    L, R = _rand(rng, m, m, m), _rand(rng, m, m, m)
    M = O.dense_from_definition(L, R)
    for T in (0, 1, 7):
        x = _rand(rng, T, m * m)
        y = O.fwd(x, L, R)
        assert y.shape == (T, m * m)
        assert np.allclose(y, x @ M.T, atol=1e-12)


def test_parameter_count():
    # Section 3.2.2: a Monarch matrix has 2 n sqrt(n) parameters.
    m = 8
    n = m * m
    assert 2 * m * m * m == 2 * n * int(math.isqrt(n))


# ------------------------------------------------------------------ backward

def _loss(x, dy, L, R):
    return float(np.sum(dy * (x @ O.dense_from_definition(L, R).T)))


def test_gradients_by_finite_differences():
    rng = np.random.default_rng(8)
    m, T = 3, 4
    n = m * m
    x, dy = _rand(rng, T, n), _rand(rng, T, n)
    L, R = _rand(rng, m, m, m), _rand(rng, m, m, m)
    g = O.bwd(x, dy, L, R)
    h = 1e-6

    def fd(arr, which):
        out = np.zeros_like(arr)
        it = np.nditer(arr, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            ap, am = arr.copy(), arr.copy()
            ap[idx] += h
            am[idx] -= h
            args_p = {"x": x, "L": L, "R": R}
            args_m = dict(args_p)
            args_p[which] = ap
            args_m[which] = am
            out[idx] = (_loss(args_p["x"], dy, args_p["L"], args_p["R"])
                        - _loss(args_m["x"], dy, args_m["L"], args_m["R"])) / (2 * h)
        return out

    assert np.allclose(g["dx"], fd(x, "x"), rtol=1e-7, atol=1e-7)
    assert np.allclose(g["dL"], fd(L, "L"), rtol=1e-7, atol=1e-7)
    assert np.allclose(g["dR"], fd(R, "R"), rtol=1e-7, atol=1e-7)


@pytest.mark.parametrize("m", [2, 4, 8])
def test_gradients_via_dense_chain_rule(m):
    # dx = M^T dy;  dM = sum_t dy_t x_t^T;  by Eq. (2)
    # dL[j,l,k] = sum_i dM[l m+j, k m+i] R[k,j,i],  dR[k,j,i] = sum_l dM[..] L[j,l,k].
    rng = np.random.default_rng(9)
    n = m * m
    T = 6
    x, dy = _rand(rng, T, n), _rand(rng, T, n)
    L, R = _rand(rng, m, m, m), _rand(rng, m, m, m)
    g = O.bwd(x, dy, L, R)
    M = O.dense_from_definition(L, R)
    assert np.allclose(g["dx"], dy @ M, atol=1e-11)
    dM4 = (dy.T @ x).reshape(m, m, m, m)                     # [l, j, k, i]
    assert np.allclose(g["dL"], np.einsum("ljki,kji->jlk", dM4, R), atol=1e-11)
    assert np.allclose(g["dR"], np.einsum("ljki,jlk->kji", dM4, L), atol=1e-11)


def test_adjoint_and_euler_identities():
    rng = np.random.default_rng(11)
    m, T = 8, 9
    n = m * m
    x, dy = _rand(rng, T, n), _rand(rng, T, n)
    L, R = _rand(rng, m, m, m), _rand(rng, m, m, m)
    y = O.fwd(x, L, R)
    g = O.bwd(x, dy, L, R)
    s = np.sum(dy * y)
    assert np.isclose(np.sum(g["dx"] * x), s, rtol=1e-12)     # <M^T dy, x> = <dy, Mx>
    assert np.isclose(np.sum(g["dL"] * L), s, rtol=1e-12)     # y is linear in L
    assert np.isclose(np.sum(g["dR"] * R), s, rtol=1e-12)     # and in R


def test_bwd_partial_outputs_and_empty():
    rng = np.random.default_rng(12)
    m = 4
    n = m * m
    x, dy = _rand(rng, 5, n), _rand(rng, 5, n)
    L, R = _rand(rng, m, m, m), _rand(rng, m, m, m)
    full = O.bwd(x, dy, L, R)
    only = O.bwd(x, dy, L, R, want=("dR",))
    assert set(only) == {"dR"} and np.array_equal(only["dR"], full["dR"])
    z = O.bwd(x[:0], dy[:0], L, R)
    assert z["dx"].shape == (0, n) and not z["dL"].any() and not z["dR"].any()


# ------------------------------------------------------------------ projection

@pytest.mark.parametrize("m", [2, 3, 4, 6])
def test_projection_recovers_monarch(m):
    # Section 3.3: if A is Monarch, Algorithm 1 recovers factors with A = P L P^T R.
    rng = np.random.default_rng(13)
    L, R = _rand(rng, m, m, m), _rand(rng, m, m, m)
    A = O.dense(L, R)
    L2, R2 = O.project(A, m)
    assert np.allclose(O.dense(L2, R2), A, atol=1e-12)
    assert np.allclose(O.dense_from_definition(L2, R2), A, atol=1e-12)
    for j in range(m):
        for k in range(m):
            s = np.linalg.svd(A.reshape(m, m, m, m)[:, j, k, :], compute_uv=False)
            assert s[1] <= 1e-12 * max(s[0], 1.0)


@pytest.mark.parametrize("m", [3, 4])
def test_projection_residual_is_discarded_spectrum(m):
    # Proof of Theorem 1: the objective splits over the m*m slices, each solved
    # by its best rank-1 approximation (Eckart-Young).
    rng = np.random.default_rng(14)
    n = m * m
    A = _rand(rng, n, n)
    L, R = O.project(A, m)
    res = np.sum((A - O.dense(L, R)) ** 2)
    A4 = A.reshape(m, m, m, m)
    tail = 0.0
    for j in range(m):
        for k in range(m):
            s = np.linalg.svd(A4[:, j, k, :], compute_uv=False)
            tail += np.sum(s[1:] ** 2)
    assert np.isclose(res, tail, rtol=1e-10)
    for _ in range(20):                                       # local optimality
        Lp = L + 1e-3 * _rand(rng, m, m, m)
        Rp = R + 1e-3 * _rand(rng, m, m, m)
        assert np.sum((A - O.dense(Lp, Rp)) ** 2) >= res - 1e-12


# ------------------------------------------------------------------ MLP block

def _gelu(a):
    return np.array([0.5 * v * (1.0 + math.erf(v / math.sqrt(2.0))) for v in a.ravel()]).reshape(a.shape)


def test_gelu_textbook_values():
    tab = _read_table("gelu_values.txt")
    m = 2
    n = 4
    I = np.stack([np.eye(m)] * m)
    for a, g in tab:
        x = np.full((1, n), a)
        h = O.mlp_fwd(x, I, I, np.zeros(n), I, I, np.zeros(n))
        assert np.allclose(h, g, rtol=1e-14, atol=1e-16)


def test_mlp_special_cases():
    rng = np.random.default_rng(15)
    m, T = 4, 5
    n = m * m
    x = _rand(rng, T, n)
    b1, b2 = _rand(rng, n), _rand(rng, n)
    I = np.stack([np.eye(m)] * m)
    Z = np.zeros((m, m, m))
    W = [_rand(rng, m, m, m) for _ in range(4)]
    # second matrix zero: y = b2
    assert np.allclose(O.mlp_fwd(x, W[0], W[1], b1, Z, W[3], b2), np.broadcast_to(b2, (T, n)))
    # identities: y = GELU(x + b1) + b2
    assert np.allclose(O.mlp_fwd(x, I, I, b1, I, I, b2), _gelu(x + b1) + b2, atol=1e-14)
    # general: composition through the dense matrices of Definition 3.1
    M1 = O.dense_from_definition(W[0], W[1])
    M2 = O.dense_from_definition(W[2], W[3])
    ref = _gelu(x @ M1.T + b1) @ M2.T + b2
    assert np.allclose(O.mlp_fwd(x, W[0], W[1], b1, W[2], W[3], b2), ref, atol=1e-11)
    # odd part of GELU: GELU(a) - GELU(-a) = a
    a = _rand(rng, 1, n)
    gp = O.mlp_fwd(a, I, I, np.zeros(n), I, I, np.zeros(n))
    gm = O.mlp_fwd(-a, I, I, np.zeros(n), I, I, np.zeros(n))
    assert np.allclose(gp - gm, a, atol=1e-14)


def _mlp_args(rng, m, T):
    n = m * m
    x, dy = _rand(rng, T, n), _rand(rng, T, n)
    W = [_rand(rng, m, m, m) / math.sqrt(m) for _ in range(4)]
    b1, b2 = 0.3 * _rand(rng, n), 0.3 * _rand(rng, n)
    return x, dy, W, b1, b2


@pytest.mark.parametrize("m", [2, 4])
def test_mlp_gradients_by_finite_differences(m):
    # f = <dy, y(x, L1, R1, b1, L2, R2, b2)>; central differences of the pinned forward.
    rng = np.random.default_rng(21)
    x, dy, W, b1, b2 = _mlp_args(rng, m, 3)
    g = O.mlp_bwd(x, dy, W[0], W[1], b1, W[2], W[3])
    args = {"x": x, "L1": W[0], "R1": W[1], "b1": b1, "L2": W[2], "R2": W[3], "b2": b2}

    def f():
        return np.sum(dy * O.mlp_fwd(args["x"], args["L1"], args["R1"], args["b1"], args["L2"],
                                     args["R2"], args["b2"]))

    h = 1e-6
    for name, key in [("x", "dx"), ("L1", "dL1"), ("R1", "dR1"), ("b1", "db1"), ("L2", "dL2"),
                      ("R2", "dR2"), ("b2", "db2")]:
        v = args[name]
        num = np.zeros_like(v)
        it = np.nditer(v, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            keep = v[idx]
            v[idx] = keep + h
            fp = f()
            v[idx] = keep - h
            fm = f()
            v[idx] = keep
            num[idx] = (fp - fm) / (2 * h)
        assert np.allclose(g[key], num, rtol=1e-6, atol=1e-7), name


def test_mlp_gradients_special_cases():
    rng = np.random.default_rng(22)
    m, T = 4, 6
    n = m * m
    x, dy, W, b1, b2 = _mlp_args(rng, m, T)
    I = np.stack([np.eye(m)] * m)
    # identities: y = GELU(x + b1) + b2, so dx = dy * GELU'(x + b1) with the derivative taken
    # numerically from the textbook-pinned GELU, and db1 = sum_t dx, db2 = sum_t dy.
    g = O.mlp_bwd(x, dy, I, I, b1, I, I)
    e = 1e-6
    dgelu = (_gelu(x + b1 + e) - _gelu(x + b1 - e)) / (2 * e)
    assert np.allclose(g["dx"], dy * dgelu, atol=1e-8)
    assert np.allclose(g["db1"], (dy * dgelu).sum(0), atol=1e-8)
    assert np.allclose(g["db2"], dy.sum(0), atol=1e-12)
    # GELU'(0) = 1/2: zero first layer and zero bias give da = dh / 2, dx = 0
    Z = np.zeros((m, m, m))
    g = O.mlp_bwd(x, dy, Z, Z, np.zeros(n), W[2], W[3])
    M2 = O.dense_from_definition(W[2], W[3])
    assert np.allclose(g["db1"], 0.5 * (dy @ M2).sum(0), atol=1e-11)
    assert not g["dx"].any() and not g["dL2"].any() and not g["dR2"].any()
    # general: chain rule through the dense matrices of Definition 3.1
    M1 = O.dense_from_definition(W[0], W[1])
    a = x @ M1.T + b1
    dgelu = (_gelu(a + e) - _gelu(a - e)) / (2 * e)
    da = (dy @ M2) * dgelu
    g = O.mlp_bwd(x, dy, W[0], W[1], b1, W[2], W[3])
    assert np.allclose(g["dx"], da @ M1, atol=1e-7)
    # second layer: the plain Monarch adjoints with input h; Euler identity <dL2, L2> = <dy, y - b2>
    y = O.mlp_fwd(x, W[0], W[1], b1, W[2], W[3], b2)
    s = np.sum(dy * (y - b2))
    assert np.isclose(np.sum(g["dL2"] * W[2]), s, rtol=1e-12)
    assert np.isclose(np.sum(g["dR2"] * W[3]), s, rtol=1e-12)
    # first layer: <dL1, L1> = <dR1, R1> = <da, a - b1>
    s1 = np.sum(da * (a - b1))
    assert np.isclose(np.sum(g["dL1"] * W[0]), s1, rtol=1e-6)
    assert np.isclose(np.sum(g["dR1"] * W[1]), s1, rtol=1e-6)


def test_mlp_bwd_empty():
    rng = np.random.default_rng(23)
    m = 4
    x, dy, W, b1, b2 = _mlp_args(rng, m, 2)
    g = O.mlp_bwd(x[:0], dy[:0], W[0], W[1], b1, W[2], W[3])
    assert g["dx"].shape == (0, m * m)
    assert not any(g[k].any() for k in ("dL1", "dR1", "db1", "dL2", "dR2", "db2"))


# ------------------------------------------------------------------ general / rectangular class

RECT = [(2, 3, 4, 5), (4, 2, 3, 2), (3, 3, 3, 3), (1, 4, 2, 3), (5, 1, 2, 4), (2, 6, 1, 3)]   # (q, b1, b, r)


@pytest.mark.parametrize("q,b1,b,r", RECT)
def test_rect_matches_definition(q, b1, b, r):
    # y = L R x with both factors materialised from the appendix's definitions
    rng = np.random.default_rng(31)
    R, Lp = _rand(rng, q, b, b1), _rand(rng, b, r, q)
    x = _rand(rng, 4, q * b1)
    Ld, Rd = O.rect_factors_from_definition(Lp, R)
    assert np.allclose(O.rect_fwd(x, Lp, R), x @ (Ld @ Rd).T, atol=1e-12)
    # parameter counts stated with the definitions: n1*b2 for R, n2*n3/b for L (b2 = b3 = b)
    assert np.count_nonzero(Rd) == q * b1 * b and np.count_nonzero(Ld) == (q * b) * (r * b) // b


@pytest.mark.parametrize("q,b1,b,r", RECT)
def test_rect_block_diagonalisation_theorem(q, b1, b, r):
    # P_(b,n3) L P_(b,n2)^T is block diagonal with b blocks of size r x q, block j = Lp[j]
    rng = np.random.default_rng(32)
    R, Lp = _rand(rng, q, b, b1), _rand(rng, b, r, q)
    Ld, _ = O.rect_factors_from_definition(Lp, R)
    n2, n3 = q * b, r * b
    Rp = O.perm_matrix_general(b, n3) @ Ld @ O.perm_matrix_general(b, n2).T
    ref = np.zeros((n3, n2))
    for j in range(b):
        ref[j * r:(j + 1) * r, j * q:(j + 1) * q] = Lp[j]
    assert np.array_equal(Rp, ref)


@pytest.mark.parametrize("b,n", [(2, 6), (3, 12), (4, 16), (1, 5), (5, 5)])
def test_general_permutation_inverse(b, n):
    # sigma_(b,n)^-1 = sigma_(n/b,n), hence P_(b,n)^T = P_(n/b,n)
    assert all(O.sigma(n // b, n, O.sigma(b, n, i)) == i for i in range(n))
    assert np.array_equal(O.perm_matrix_general(b, n).T, O.perm_matrix_general(n // b, n))


@pytest.mark.parametrize("m", [2, 3, 5])
def test_rect_reduces_to_square(m):
    rng = np.random.default_rng(33)
    L, R = _rand(rng, m, m, m), _rand(rng, m, m, m)
    x = _rand(rng, 3, m * m)
    assert np.allclose(O.rect_fwd(x, L, R), O.fwd(x, L, R), atol=1e-13)
    assert np.allclose(O.rect_fwd(x, L, R), x @ O.dense_from_definition(L, R).T, atol=1e-12)
    assert np.array_equal(O.perm_matrix_general(m, m * m), O.perm_matrix(m))


def test_rect_kronecker_closed_form():
    # every R_k = B (b x b1) and every diagonal-block pattern equal (Lp[j] = A, r x q): M = A kron B
    rng = np.random.default_rng(34)
    q, b1, b, r = 3, 4, 2, 5
    A, B = _rand(rng, r, q), _rand(rng, b, b1)
    x = _rand(rng, 6, q * b1)
    y = O.rect_fwd(x, np.stack([A] * b), np.stack([B] * q))
    assert np.allclose(y, x @ np.kron(A, B).T, atol=1e-12)
    # identity blocks on a square instance give the identity matrix (the class contains I)
    n = 12
    y = O.rect_fwd(x, np.stack([np.eye(3)] * 4), np.stack([np.eye(4)] * 3))
    assert np.allclose(y, x)
    assert y.shape == (6, n)


# ------------------------------------------------------------------ complex factors (Section 3.2: FFT, MM*)

def _crand(rng, *shape):
    return rng.standard_normal(shape) + 1j * rng.standard_normal(shape)


@pytest.mark.parametrize("m", [2, 3, 4])
def test_cplx_routes_agree_and_reduce_to_real(m):
    rng = np.random.default_rng(41)
    n = m * m
    L, R, x = _crand(rng, m, m, m), _crand(rng, m, m, m), _crand(rng, 5, n)
    M = O.cplx_dense_from_definition(L, R)
    assert np.allclose(O.cplx_fwd(x, L, R), x @ M.T, atol=1e-12)
    assert np.allclose(O.cplx_fwd(x, L, R, adjoint=True), x @ M.conj(), atol=1e-12)      # rows of x times M^H^T
    # real data through the complex route equals the (pinned) real oracle
    assert np.allclose(O.cplx_fwd(x.real, L.real, R.real).real, O.fwd(x.real, L.real, R.real), atol=1e-12)
    assert np.allclose(O.cplx_fwd(x.real, L.real, R.real, adjoint=True).real,
                       O.bwd(x.real, x.real, L.real, R.real, want=("dx",))["dx"], atol=1e-12)
    # <M x, y> = <x, M^H y>
    y = _crand(rng, 5, n)
    lhs = np.sum(O.cplx_fwd(x, L, R) * y.conj())
    rhs = np.sum(x * O.cplx_fwd(y, L, R, adjoint=True).conj())
    assert np.isclose(lhs, rhs, rtol=1e-12)


@pytest.mark.parametrize("m", [2, 4, 8])
def test_dft_is_monarch(m):
    # Section 3.2: the DFT matrix (times the stated permutation) is a Monarch matrix; numpy.fft is the pin
    rng = np.random.default_rng(42)
    n = m * m
    L, R = O.dft_factors(m)
    x = _crand(rng, 3, n)
    xp = x.reshape(3, m, m).transpose(0, 2, 1).reshape(3, n)              # P x
    assert np.allclose(O.cplx_fwd(xp, L, R), np.fft.fft(x, axis=1), atol=1e-10)
    # F_n F_n^H = n I: the MM* product of the DFT factors with themselves
    z = O.cplx_fwd(O.cplx_fwd(x, L, R, adjoint=True), L, R)
    assert np.allclose(z, n * x, atol=1e-9)


@pytest.mark.parametrize("q,b1,b,r", [(2, 3, 4, 5), (4, 2, 3, 2), (3, 3, 3, 3), (1, 4, 2, 3)])
def test_rect_gradients(q, b1, b, r):
    rng = np.random.default_rng(35)
    T = 4
    R, Lp = _rand(rng, q, b, b1), _rand(rng, b, r, q)
    x, dy = _rand(rng, T, q * b1), _rand(rng, T, r * b)
    g = O.rect_bwd(x, dy, Lp, R)
    # dx = M^T dy with M from the definitions' dense factors
    Ld, Rd = O.rect_factors_from_definition(Lp, R)
    assert np.allclose(g["dx"], dy @ (Ld @ Rd), atol=1e-12)
    # central differences of f = <dy, L R x> in the parameters
    args = {"L": Lp, "R": R}
    h = 1e-6
    for name, key in (("L", "dL"), ("R", "dR")):
        v = args[name]
        num = np.zeros_like(v)
        it = np.nditer(v, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            keep = v[idx]
            v[idx] = keep + h
            fp = np.sum(dy * O.rect_fwd(x, args["L"], args["R"]))
            v[idx] = keep - h
            fm = np.sum(dy * O.rect_fwd(x, args["L"], args["R"]))
            v[idx] = keep
            num[idx] = (fp - fm) / (2 * h)
        assert np.allclose(g[key], num, rtol=1e-7, atol=1e-7), name
    # Euler identities (y is bilinear in the two factors) and the adjoint identity
    s = np.sum(dy * O.rect_fwd(x, Lp, R))
    assert np.isclose(np.sum(g["dL"] * Lp), s, rtol=1e-12) and np.isclose(np.sum(g["dR"] * R), s, rtol=1e-12)
    assert np.isclose(np.sum(g["dx"] * x), s, rtol=1e-12)


WRAPPED = [(3, 2, 2, 4, 2), (2, 3, 4, 2, 3), (2, 2, 3, 5, 2), (3, 1, 5, 3, 2), (2, 4, 2, 6, 1), (2, 2, 6, 2, 3),
           (1, 3, 4, 4, 2)]


@pytest.mark.parametrize("q,b1,b2,b3,r", WRAPPED)
def test_wrapped_rect_matches_definition(q, b1, b2, b3, r):
    """The two-step multiply against L R x with both factors materialised from the appendix's rectangular definition
    (block-diagonal R; L a grid of wrapped-diagonal blocks, whose zero pattern is tested entry by entry), and the
    number of stored entries against the count the paper states, n2 n3 / min(b2, b3)."""
    rng = np.random.default_rng(q * 1000 + b1 * 100 + b2 * 10 + b3)
    R = rng.standard_normal((q, b2, b1)); Lw = rng.standard_normal((r, q, max(b2, b3)))
    x = rng.standard_normal((5, q * b1))
    Ld, Rd = O.rectw_factors_from_definition(Lw, R, b3)
    assert np.count_nonzero(Ld) == (q * b2) * (r * b3) // min(b2, b3) == Lw.size
    assert np.allclose(O.rectw_fwd(x, Lw, R, b3), x @ (Ld @ Rd).T, atol=1e-12)


@pytest.mark.parametrize("q,b1,b,r", [(3, 2, 4, 2), (2, 5, 3, 3)])
def test_wrapped_rect_reduces_to_diagonal_blocks(q, b1, b, r):
    """b2 = b3: a wrapped diagonal is a diagonal, and the multiply is the rectangular multiply pinned above with
    Lp[j, l, k] = Lw[l, k, j]."""
    rng = np.random.default_rng(77 + q + b)
    R = rng.standard_normal((q, b, b1)); Lw = rng.standard_normal((r, q, b)); x = rng.standard_normal((4, q * b1))
    Lp = np.ascontiguousarray(Lw.transpose(2, 0, 1))
    assert np.allclose(O.rectw_fwd(x, Lw, R, b), O.rect_fwd(x, Lp, R), atol=1e-12)
    dy = rng.standard_normal((4, r * b))
    g, h = O.rectw_bwd(x, dy, Lw, R, b), O.rect_bwd(x, dy, Lp, R)
    assert np.allclose(g["dx"], h["dx"], atol=1e-12) and np.allclose(g["dR"], h["dR"], atol=1e-12)
    assert np.allclose(g["dL"], h["dL"].transpose(1, 2, 0), atol=1e-12)


@pytest.mark.parametrize("q,b1,b2,b3,r", WRAPPED)
def test_wrapped_rect_gradients(q, b1, b2, b3, r):
    """dx, dL, dR against the dense chain rule through the factors of the definition (dM = dy^T x, dL = dM R^T and
    dR = L^T dM restricted to the stored entries) and central differences of the pinned forward."""
    rng = np.random.default_rng(5000 + q * 100 + b2 * 10 + b3)
    R = rng.standard_normal((q, b2, b1)); Lw = rng.standard_normal((r, q, max(b2, b3)))
    x = rng.standard_normal((6, q * b1)); dy = rng.standard_normal((6, r * b3))
    g = O.rectw_bwd(x, dy, Lw, R, b3)
    Ld, Rd = O.rectw_factors_from_definition(Lw, R, b3)
    assert np.allclose(g["dx"], dy @ (Ld @ Rd), atol=1e-12)
    dM = dy.T @ x
    dLd, dRd = dM @ Rd.T, Ld.T @ dM
    i0, j0 = O.wrapped_positions(b2, b3)
    for l in range(r):
        for k in range(q):
            assert np.allclose(g["dL"][l, k], dLd[l * b3 + i0, k * b2 + j0], atol=1e-11)
    for k in range(q):
        assert np.allclose(g["dR"][k], dRd[k * b2:(k + 1) * b2, k * b1:(k + 1) * b1], atol=1e-11)
    f = lambda Lw_, R_: float(np.sum(dy * O.rectw_fwd(x, Lw_, R_, b3)))
    eps = 1e-6
    for idx in [(0, 0, 0), (r - 1, q - 1, max(b2, b3) - 1)]:
        d = np.zeros_like(Lw); d[idx] = eps
        assert abs((f(Lw + d, R) - f(Lw - d, R)) / (2 * eps) - g["dL"][idx]) < 1e-6
    for idx in [(0, 0, 0), (q - 1, b2 - 1, b1 - 1)]:
        d = np.zeros_like(R); d[idx] = eps
        assert abs((f(Lw, R + d) - f(Lw, R - d)) / (2 * eps) - g["dR"][idx]) < 1e-6


def test_rect_gradients_reduce_to_square():
    rng = np.random.default_rng(36)
    m, T = 4, 5
    L, R = _rand(rng, m, m, m), _rand(rng, m, m, m)
    x, dy = _rand(rng, T, m * m), _rand(rng, T, m * m)
    g, ref = O.rect_bwd(x, dy, L, R), O.bwd(x, dy, L, R)
    for k in ("dx", "dL", "dR"):
        assert np.allclose(g[k], ref[k], atol=1e-12), k
