"""CPU oracle for the Monarch multiply (Dao et al., arXiv 2204.00595).

TEST INFRASTRUCTURE ONLY.  Nothing in the product path may import this
module: it exists so that tests, the smoke check and the benchmark's CPU
baseline can compare the CUDA library against a plain fp64 statement of the
paper's definitions.  It shares no code with the CUDA library.

Two layers:

* ``monarch_oracle.c`` - plain C loops in fp64 over the paper's multiply
  steps (Section 3.3, steps 1-3), their adjoints, the entry formula Eq. (2)
  and the Monarch feed-forward block with its gradients.  Compiled on demand
  with gcc.
* numpy routines in this file that restate *Definition 3.1 literally*
  (explicit permutation and block-diagonal matrices) and Algorithm 1
  (projection by rank-1 SVDs).  They are the independent routes the C loops
  are pinned against; they only run at tiny n.

All inputs and outputs are float64, C-contiguous:
  x, y, dy, dx : [T, n]      L, R : [m, m, m] = [block, out, in]     n = m*m
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import sys

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "monarch_oracle.c")
_LIB = os.path.join(_HERE, "libmonarch_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle (gcc -O2 -fopenmp) next to its source."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_fwd.restype = ctypes.c_int
        lib.oracle_fwd.argtypes = [dp, dp, dp, dp, dp, ctypes.c_long, ctypes.c_int]
        lib.oracle_dense.restype = None
        lib.oracle_dense.argtypes = [dp, dp, dp, ctypes.c_int]
        lib.oracle_bwd.restype = ctypes.c_int
        lib.oracle_bwd.argtypes = [dp] * 7 + [ctypes.c_long, ctypes.c_int]
        lib.oracle_mlp_fwd.restype = ctypes.c_int
        lib.oracle_mlp_fwd.argtypes = [dp] * 8 + [ctypes.c_long, ctypes.c_int]
        lib.oracle_rect_fwd.restype = ctypes.c_int
        lib.oracle_rect_fwd.argtypes = [dp] * 4 + [ctypes.c_long] + [ctypes.c_int] * 4
        lib.oracle_rect_bwd.restype = ctypes.c_int
        lib.oracle_rect_bwd.argtypes = [dp] * 7 + [ctypes.c_long] + [ctypes.c_int] * 4
        lib.oracle_mlp_bwd.restype = ctypes.c_int
        lib.oracle_mlp_bwd.argtypes = [dp] * 14 + [ctypes.c_long, ctypes.c_int]
        _lib = lib
    return _lib


def num_threads() -> int:
    """Host threads the C loops will use (OpenMP's max threads)."""
    return int(_load().oracle_num_threads())


def _f64(a, shape=None):
    a = np.ascontiguousarray(a, dtype=np.float64)
    if shape is not None and tuple(a.shape) != tuple(shape):
        raise ValueError(f"expected shape {shape}, got {a.shape}")
    return a


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _m_of(L):
    m = L.shape[0]
    if L.shape != (m, m, m):
        raise ValueError("weights must be [m, m, m]")
    return m


# --------------------------------------------------------------------------
# C loops: steps 1-3, adjoints, Eq. (2), feed-forward block
# --------------------------------------------------------------------------

def fwd(x, L, R, return_u: bool = False):
    """y = M x by the paper's steps 1-3 (Section 3.3).  x: [T, n]."""
    L = _f64(L); R = _f64(R); m = _m_of(L); n = m * m
    x = _f64(x); T = x.shape[0]
    if x.shape != (T, n) or R.shape != L.shape:
        raise ValueError("shape mismatch")
    y = np.empty((T, n), dtype=np.float64)
    u = np.empty((T, n), dtype=np.float64) if return_u else None
    if _load().oracle_fwd(_p(x), _p(L), _p(R), _p(y), _p(u), T, m):
        raise MemoryError("oracle_fwd")
    return (y, u.reshape(T, m, m)) if return_u else y


def dense(L, R):
    """The n x n matrix M by the entry formula Eq. (2)."""
    L = _f64(L); R = _f64(R); m = _m_of(L); n = m * m
    M = np.empty((n, n), dtype=np.float64)
    _load().oracle_dense(_p(L), _p(R), _p(M), m)
    return M


def bwd(x, dy, L, R, want=("dx", "dL", "dR")):
    """Adjoints of steps 1-3 for f = <dy, Mx>: returns dict with dx, dL, dR."""
    L = _f64(L); R = _f64(R); m = _m_of(L); n = m * m
    x = _f64(x); dy = _f64(dy); T = x.shape[0]
    if x.shape != (T, n) or dy.shape != (T, n):
        raise ValueError("shape mismatch")
    out = {}
    if "dx" in want:
        out["dx"] = np.empty((T, n), dtype=np.float64)
    if "dL" in want:
        out["dL"] = np.empty((m, m, m), dtype=np.float64)
    if "dR" in want:
        out["dR"] = np.empty((m, m, m), dtype=np.float64)
    if _load().oracle_bwd(_p(x), _p(dy), _p(L), _p(R), _p(out.get("dx")),
                          _p(out.get("dL")), _p(out.get("dR")), T, m):
        raise MemoryError("oracle_bwd")
    return out


def mlp_fwd(x, L1, R1, b1, L2, R2, b2):
    """y = M2 GELU(M1 x + b1) + b2 with the erf form of GELU."""
    L1 = _f64(L1); R1 = _f64(R1); L2 = _f64(L2); R2 = _f64(R2)
    m = _m_of(L1); n = m * m
    b1 = _f64(b1, (n,)); b2 = _f64(b2, (n,))
    x = _f64(x); T = x.shape[0]
    y = np.empty((T, n), dtype=np.float64)
    if _load().oracle_mlp_fwd(_p(x), _p(L1), _p(R1), _p(b1), _p(L2), _p(R2), _p(b2),
                              _p(y), T, m):
        raise MemoryError("oracle_mlp_fwd")
    return y


def mlp_bwd(x, dy, L1, R1, b1, L2, R2):
    """Gradients of <dy, y> for y = M2 GELU(M1 x + b1) + b2 (chain rule through the block).

    Returns dict with dx [T, n], dL1, dR1, dL2, dR2 [m, m, m], db1, db2 [n].
    """
    L1 = _f64(L1); R1 = _f64(R1); L2 = _f64(L2); R2 = _f64(R2)
    m = _m_of(L1); n = m * m
    b1 = _f64(b1, (n,))
    x = _f64(x); dy = _f64(dy); T = x.shape[0]
    if x.shape != (T, n) or dy.shape != (T, n):
        raise ValueError("shape mismatch")
    out = {"dx": np.empty((T, n))}
    for k in ("dL1", "dR1", "dL2", "dR2"):
        out[k] = np.empty((m, m, m))
    out["db1"] = np.empty(n)
    out["db2"] = np.empty(n)
    if _load().oracle_mlp_bwd(_p(x), _p(dy), _p(L1), _p(R1), _p(b1), _p(L2), _p(R2), _p(out["dx"]),
                              _p(out["dL1"]), _p(out["dR1"]), _p(out["db1"]), _p(out["dL2"]),
                              _p(out["dR2"]), _p(out["db2"]), T, m):
        raise MemoryError("oracle_mlp_bwd")
    return out


def rect_fwd(x, Lp, R):
    """y = L R x for the general (rectangular) Monarch class of the appendix.

    R: [q, b, b1] (q blocks of b x b1), Lp: [b, r, q] with Lp[j, l, k] = S_{l,k}[j, j] (the diagonal
    blocks of L gathered into the b blocks of its block-diagonal form), x: [T, q*b1] -> y: [T, r*b].
    """
    Lp = _f64(Lp); R = _f64(R)
    q, b, b1 = R.shape
    if Lp.ndim != 3 or Lp.shape[0] != b or Lp.shape[2] != q:
        raise ValueError("Lp must be [b, r, q] for R of shape [q, b, b1]")
    r = Lp.shape[1]
    x = _f64(x); T = x.shape[0]
    if x.shape != (T, q * b1):
        raise ValueError("x must be [T, q*b1]")
    y = np.empty((T, r * b), dtype=np.float64)
    if _load().oracle_rect_fwd(_p(x), _p(Lp), _p(R), _p(y), T, q, b1, b, r):
        raise MemoryError("oracle_rect_fwd")
    return y


def rect_bwd(x, dy, Lp, R):
    """Gradients of <dy, L R x> for the general (rectangular) class: dict with dx, dL (like Lp), dR."""
    Lp = _f64(Lp); R = _f64(R)
    q, b, b1 = R.shape
    r = Lp.shape[1]
    x = _f64(x); dy = _f64(dy); T = x.shape[0]
    if x.shape != (T, q * b1) or dy.shape != (T, r * b) or Lp.shape != (b, r, q):
        raise ValueError("shape mismatch")
    out = {"dx": np.empty((T, q * b1)), "dL": np.empty((b, r, q)), "dR": np.empty((q, b, b1))}
    if _load().oracle_rect_bwd(_p(x), _p(dy), _p(Lp), _p(R), _p(out["dx"]), _p(out["dL"]), _p(out["dR"]),
                               T, q, b1, b, r):
        raise MemoryError("oracle_rect_bwd")
    return out


# --------------------------------------------------------------------------
# numpy restatements of the definitions (tiny n only)
# --------------------------------------------------------------------------

def perm_matrix(m: int) -> np.ndarray:
    """The permutation P of Definition 3.1 as an n x n 0/1 matrix.

    P maps [x_1..x_n] to [x_1, x_{1+m}, ..., x_{1+(m-1)m}, x_2, ...]: output
    position a*m+b holds input element b*m+a (0-indexed) - reshape to m x m,
    transpose, flatten.
    """
    n = m * m
    P = np.zeros((n, n), dtype=np.float64)
    for a in range(m):
        for b in range(m):
            P[a * m + b, b * m + a] = 1.0
    return P


def blockdiag(W) -> np.ndarray:
    """diag(W_0, ..., W_{m-1}) as a dense n x n matrix."""
    W = np.asarray(W, dtype=np.float64)
    m = W.shape[0]
    n = m * m
    B = np.zeros((n, n), dtype=np.float64)
    for b in range(m):
        B[b * m:(b + 1) * m, b * m:(b + 1) * m] = W[b]
    return B


def dense_from_definition(L, R) -> np.ndarray:
    """M = P L P^T R with every factor materialised (Definition 3.1)."""
    m = np.asarray(L).shape[0]
    P = perm_matrix(m)
    return P @ blockdiag(L) @ P.T @ blockdiag(R)


def sigma(b: int, n: int, i: int) -> int:
    """The appendix's permutation sigma_(b,n): i = (i1, i0)_b  ->  (i0, i1)_{n/b} = i0 * (n/b) + i1."""
    i1, i0 = divmod(i, b)
    return i0 * (n // b) + i1


def perm_matrix_general(b: int, n: int) -> np.ndarray:
    """P_(b,n) as used in the appendix's block-diagonalisation proofs: R'[sigma(i), sigma(j)] = L[i, j]
    for R' = P L P^T, i.e. P has its ones at (sigma(i), i).  (The prose "reshape b x n/b, transpose,
    flatten" describes the transpose of this matrix; the two coincide when b = n/b.)"""
    P = np.zeros((n, n), dtype=np.float64)
    for i in range(n):
        P[sigma(b, n, i), i] = 1.0
    return P


def rect_factors_from_definition(Lp, R):
    """The two factors of the rectangular definition as dense matrices: R = diag(R_k) (n2 x n1) and L
    (n3 x n2) whose (l, k) block is the diagonal matrix S_{l,k} with S_{l,k}[j, j] = Lp[j, l, k]."""
    Lp = np.asarray(Lp, dtype=np.float64); R = np.asarray(R, dtype=np.float64)
    q, b, b1 = R.shape
    r = Lp.shape[1]
    Rd = np.zeros((q * b, q * b1))
    for k in range(q):
        Rd[k * b:(k + 1) * b, k * b1:(k + 1) * b1] = R[k]
    Ld = np.zeros((r * b, q * b))
    for l in range(r):
        for k in range(q):
            Ld[l * b:(l + 1) * b, k * b:(k + 1) * b] = np.diag(Lp[:, l, k])
    return Ld, Rd


# --------------------------------------------------------------------------
# rectangular class with wrapped-diagonal blocks (appendix, rectangular definition with b2 != b3)
# --------------------------------------------------------------------------

def wrapped_positions(b2: int, b3: int):
    """Where the stored entries of one wrapped-diagonal block S (b3 x b2) sit: entry e of the max(b2, b3) stored
    values is S[i0[e], j0[e]].  For b2 <= b3 a row i0 holds its one non-zero in column i0 mod b2; for b2 > b3 the
    definition is applied to the transpose: a column j0 holds its one non-zero in row j0 mod b3."""
    e = np.arange(max(b2, b3))
    return (e, e % b2) if b2 <= b3 else (e % b3, e)


def rectw_factors_from_definition(Lw, R, b3: int):
    """Dense factors of the rectangular definition: R = diag(R_k) (n2 x n1) and L (n3 x n2), an r x q grid of
    wrapped-diagonal blocks, built entry by entry from the definition's rule for the zero pattern (every (i, j) is
    visited and tested), with S_{l,k}'s stored values Lw[l, k, :]."""
    Lw = np.asarray(Lw, dtype=np.float64); R = np.asarray(R, dtype=np.float64)
    q, b2, b1 = R.shape
    r = Lw.shape[0]
    if Lw.shape != (r, q, max(b2, b3)):
        raise ValueError("Lw must be [r, q, max(b2, b3)]")
    Rd = np.zeros((q * b2, q * b1))
    for k in range(q):
        Rd[k * b2:(k + 1) * b2, k * b1:(k + 1) * b1] = R[k]
    Ld = np.zeros((r * b3, q * b2))
    for i in range(r * b3):
        i1, i0 = divmod(i, b3)
        for j in range(q * b2):
            j1, j0 = divmod(j, b2)
            if b2 <= b3:
                if i0 % b2 == j0:
                    Ld[i, j] = Lw[i1, j1, i0]
            elif j0 % b3 == i0:
                Ld[i, j] = Lw[i1, j1, j0]
    return Ld, Rd


def rectw_fwd(x, Lw, R, b3: int) -> np.ndarray:
    """y = L R x for the rectangular class with wrapped-diagonal blocks, as two steps:
    u[t, k, :] = R_k x[t, k, :], then every stored entry of L moves one element of u to one element of y:
    y[t, l*b3 + i0(e)] += Lw[l, k, e] * u[t, k*b2 + j0(e)].   x: [T, q*b1] -> y: [T, r*b3]."""
    Lw = _f64(Lw); R = _f64(R); x = _f64(x)
    q, b2, b1 = R.shape
    r = Lw.shape[0]
    T = x.shape[0]
    if Lw.shape != (r, q, max(b2, b3)) or x.shape != (T, q * b1):
        raise ValueError("shape mismatch")
    i0, j0 = wrapped_positions(b2, b3)
    u = np.einsum("kji,tki->tkj", R, x.reshape(T, q, b1))
    y = np.zeros((T, r, b3))
    for l in range(r):
        for k in range(q):
            np.add.at(y[:, l, :], (slice(None), i0), Lw[l, k][None, :] * u[:, k, j0])
    return y.reshape(T, r * b3)


def rectw_bwd(x, dy, Lw, R, b3: int):
    """Gradients of <dy, L R x> for the wrapped-diagonal rectangular class: dict with dx, dL (like Lw), dR."""
    Lw = _f64(Lw); R = _f64(R); x = _f64(x); dy = _f64(dy)
    q, b2, b1 = R.shape
    r = Lw.shape[0]
    T = x.shape[0]
    if Lw.shape != (r, q, max(b2, b3)) or x.shape != (T, q * b1) or dy.shape != (T, r * b3):
        raise ValueError("shape mismatch")
    i0, j0 = wrapped_positions(b2, b3)
    xk = x.reshape(T, q, b1)
    u = np.einsum("kji,tki->tkj", R, xk)
    dyl = dy.reshape(T, r, b3)
    du = np.zeros((T, q, b2))
    dL = np.empty_like(Lw)
    for l in range(r):
        for k in range(q):
            np.add.at(du[:, k, :], (slice(None), j0), Lw[l, k][None, :] * dyl[:, l, i0])
            dL[l, k] = np.einsum("te,te->e", dyl[:, l, i0], u[:, k, j0])
    return {"dx": np.einsum("kji,tkj->tki", R, du).reshape(T, q * b1), "dL": dL,
            "dR": np.einsum("tkj,tki->kji", du, xk)}


def cplx_dense_from_definition(L, R) -> np.ndarray:
    """Definition 3.1 with complex factors: M = P L P^T R as a dense complex n x n matrix."""
    L = np.asarray(L, dtype=np.complex128); R = np.asarray(R, dtype=np.complex128)
    m = L.shape[0]
    n = m * m
    P = perm_matrix(m)
    Ld = np.zeros((n, n), dtype=np.complex128)
    Rd = np.zeros((n, n), dtype=np.complex128)
    for b in range(m):
        Ld[b * m:(b + 1) * m, b * m:(b + 1) * m] = L[b]
        Rd[b * m:(b + 1) * m, b * m:(b + 1) * m] = R[b]
    return P @ Ld @ P.T @ Rd


def cplx_fwd(x, L, R, adjoint: bool = False) -> np.ndarray:
    """Complex Monarch multiply by the paper's steps 1-3 in complex128 (x: [T, n], L, R: [m, m, m]);
    adjoint=True applies M^H = R^H P L^H P (the second factor of the MM* products of Section 3.2)."""
    x = np.asarray(x, dtype=np.complex128); L = np.asarray(L, dtype=np.complex128)
    R = np.asarray(R, dtype=np.complex128)
    m = L.shape[0]
    T = x.shape[0]
    if not adjoint:
        u = np.einsum("kji,tki->tkj", R, x.reshape(T, m, m))           # step 1
        return np.einsum("jlk,tkj->tlj", L, u).reshape(T, m * m)       # steps 2-3
    du = np.einsum("jlk,tlj->tkj", L.conj(), x.reshape(T, m, m))       # adjoint of steps 2-3
    return np.einsum("kji,tkj->tki", R.conj(), du).reshape(T, m * m)   # adjoint of step 1


def dft_factors(m: int):
    """Complex Monarch factors with M = F_n P (F_n the n-point DFT matrix, omega = exp(-2 pi i / n)): the
    Cooley-Tukey split f = f1 m + f0, s = s1 m + s0 gives L_j = F_m and R_k = diag(omega_n^{j k}) F_m."""
    n = m * m
    a = np.arange(m)
    Fm = np.exp(-2j * np.pi * np.outer(a, a) / m)
    L = np.stack([Fm] * m)
    R = np.stack([np.exp(-2j * np.pi * a * k / n)[:, None] * Fm for k in range(m)])
    return L, R


def project(A, m: int):
    """Algorithm 1: closest Monarch matrix to a dense A in Frobenius norm.

    A is viewed as A~[l, j, k, i] = A[l*m+j, k*m+i]; every slice
    A~[:, j, k, :] (an m x m matrix indexed l, i) is replaced by its best
    rank-1 approximation u v^T, with L[j, :, k] = u and R[k, j, :] = v.
    The paper fixes only the product u v^T; here both carry sqrt(sigma_1).
    """
    A = np.asarray(A, dtype=np.float64)
    n = m * m
    if A.shape != (n, n):
        raise ValueError("A must be n x n with n = m*m")
    A4 = A.reshape(m, m, m, m)            # [l, j, k, i]
    L = np.zeros((m, m, m), dtype=np.float64)
    R = np.zeros((m, m, m), dtype=np.float64)
    for j in range(m):
        for k in range(m):
            S = A4[:, j, k, :]
            U, s, Vt = np.linalg.svd(S)
            L[j, :, k] = U[:, 0] * np.sqrt(s[0])
            R[k, j, :] = Vt[0, :] * np.sqrt(s[0])
    return L, R


if __name__ == "__main__":
    build(force=True)
    print("built", _LIB, "threads", num_threads(), file=sys.stderr)
