"""CPU oracle for Draco's repetition and cyclic codes (arXiv 1803.09877).

TEST INFRASTRUCTURE ONLY.  A plain, slow, fp64 / complex128 restatement of what
the paper's encoders and decoders compute, written from the paper and sharing no
code with the CUDA path.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may call it; the product never does.

Conventions.  n = the paper's P (compute nodes, and B = P gradients), s = the
number of adversaries tolerated, r = 2 s + 1, d = gradient dimension.  Matrices
are stored worker-major: ``G[k]`` is gradient g_k, ``Z[j]`` / ``R[j]`` is what
node j sends / what the PS receives from it, i.e. the transpose of the paper's
d x P matrices.  Indices are 0-based.

Pins (tests/test_oracle_*.py): exact recovery of G 1_P for every placement of
<= s adversaries by brute force (Definition 2, Theorems 2 and 5); failure once s
is exceeded (Theorem 1); the hand-derived n=4, s=1 coefficient table; Lemma 3
(support of W, 1_P in the span); Lemma 7 (C_L C_R^dagger = 0, clean syndromes
vanish); the locator returning t = (f N)^T value for value (proof of Lemma 4);
Algorithm 2 against sort-and-count; the adversary-free decode reducing to a
plain sum; NaN / infinite vectors and five adjacent adversaries at n = 45
decoded at every placement; the colluding attack of Theorem 1's proof.

Parity unpinned (readings, not paper facts; they do not change the exact
result): the rank cutoff ``theta`` of the locator and its "rank largest |t_j|"
reading of t_j != 0; the grouping used when 2 s + 1 does not divide n; the
minimum-norm choice among the valid decode vectors b; the cutoff of the locator's
later passes (theta * scale * sum |lambda_k|).
"""
from __future__ import annotations

import functools

import mpmath
import numpy as np

# --------------------------------------------------------------------------
# Repetition code  (Section 3, "Fractional Repetition Code")
# --------------------------------------------------------------------------


def rep_groups(n: int, s: int) -> list[tuple[int, int]]:
    """Groups of consecutive workers as ``(first, size)``.

    Section 3: the allocation matrix A^Rep is block diagonal with all-ones
    r x r blocks, so nodes l r .. l r + r - 1 form group l (n / r groups).  The
    paper assumes r | n.  Reading used when it does not: floor(n / r) groups of
    consecutive workers, the first ``n mod groups`` of them one member larger;
    every group then has >= r members and still out-votes s adversaries.
    """
    r = 2 * s + 1
    if n < 1 or s < 0 or r > n:
        raise ValueError("need n >= 1, s >= 0 and 2 s + 1 <= n (Corollary of Theorem 1)")
    g = n // r
    base, extra = divmod(n, g)
    out, first = [], 0
    for ell in range(g):
        size = base + 1 if ell < extra else base
        out.append((first, size))
        first += size
    return out


def rep_allocation(n: int, s: int) -> np.ndarray:
    """A^Rep: A[j][k] = 1 iff nodes j and k are in the same group."""
    A = np.zeros((n, n), dtype=np.int64)
    for first, size in rep_groups(n, s):
        A[first:first + size, first:first + size] = 1
    return A


def rep_encode(G: np.ndarray, n: int, s: int) -> np.ndarray:
    """E^Rep_j(Y_j) = Y_j 1_P: node j sends the sum of its allocated gradients.

    Summed in fp64 in ascending gradient index (so nodes with the same
    allocation produce the same bits), then rounded to the fp32 vector sent.
    """
    A = rep_allocation(n, s)
    G64 = np.asarray(G, dtype=np.float64)
    Z = np.zeros((n, G64.shape[1]), dtype=np.float64)
    for j in range(n):
        for k in range(n):
            if A[j, k]:
                Z[j] += G64[k]
    return Z.astype(np.float32)


def majority_stream(items: np.ndarray):
    """Algorithm 2 (streaming majority vote) on every column of ``items`` at once.

    ``items`` is ``[m][L]`` of 32-bit patterns; item i of column c is
    ``items[i][c]``.  Returns the candidate ``Ma`` per column (the majority item
    whenever one exists).  Equality is equality of bit patterns.
    """
    items = np.asarray(items)
    m = items.shape[0]
    ma = items[0].copy()
    counter = np.zeros(items.shape[1], dtype=np.int64)
    for i in range(m):
        x = items[i]
        empty = counter == 0
        same = ma == x
        ma = np.where(empty, x, ma)
        counter = np.where(empty, 1, np.where(same, counter + 1, counter - 1))
    return ma


def rep_decode(R: np.ndarray, n: int, s: int) -> dict:
    """D^Rep(R) = sum over groups of Maj(group's received vectors).

    Returns
      u        fp64 ``[d]``  sum of the group majorities, groups ascending
      maj      fp32 ``[groups][d]``  the value selected for each group
      flags    bool ``[n]``  node j differs from its group's selection somewhere
      no_majority  number of (group, coordinate) pairs whose candidate is not
                   held by strictly more than half of the group
    """
    R = np.ascontiguousarray(R, dtype=np.float32)
    bits = R.view(np.uint32)
    groups = rep_groups(n, s)
    d = R.shape[1]
    u = np.zeros(d, dtype=np.float64)
    maj = np.empty((len(groups), d), dtype=np.float32)
    flags = np.zeros(n, dtype=bool)
    no_majority = 0
    for ell, (first, size) in enumerate(groups):
        block = bits[first:first + size]
        cand = majority_stream(block)
        votes = (block == cand[None, :]).sum(axis=0)
        no_majority += int(np.count_nonzero(2 * votes <= size))
        flags[first:first + size] = (block != cand[None, :]).any(axis=1)
        maj[ell] = cand.view(np.float32)
        u += maj[ell].astype(np.float64)
    return {"u": u, "maj": maj, "flags": flags, "no_majority": no_majority}


# --------------------------------------------------------------------------
# Cyclic code  (Section 3, "Cyclic Code")
# --------------------------------------------------------------------------


def idft_matrix(n: int) -> np.ndarray:
    """C[j][k] = exp(2 pi i j k / n) / sqrt(n)  (0-based form of the paper's C)."""
    jk = np.outer(np.arange(n), np.arange(n)) % n
    return np.exp(2j * np.pi * jk / n) / np.sqrt(n)


def cyc_allocation(n: int, s: int) -> np.ndarray:
    """A^Cyc: row j holds 2 s + 1 cyclically consecutive ones starting at column j."""
    if n < 1 or s < 0 or 2 * s + 1 > n:
        raise ValueError("need 2 s + 1 <= n")
    A = np.zeros((n, n), dtype=np.int64)
    for j in range(n):
        for t in range(2 * s + 1):
            A[j, (j + t) % n] = 1
    return A


def _mp_root(n: int, e: int):
    return mpmath.expjpi(mpmath.mpf(2 * (e % n)) / n)


def cyc_W_by_definition(n: int, s: int, dps: int = 60) -> np.ndarray:
    """W = [Q 1_P] C_L, with row j of Q solving [q_j 1] [C_L]_{., alpha_j} = 0.

    alpha_j = the columns where row j of A^Cyc is zero (n - 2 s - 1 of them).
    Solved in ``dps``-digit arithmetic (the Vandermonde systems are badly
    conditioned in fp64 for n in the tens), rounded to complex128 at the end.
    """
    A = cyc_allocation(n, s)
    rows = n - 2 * s                      # rows of C_L
    m = rows - 1                          # length of q_j
    with mpmath.workdps(dps):
        rt = mpmath.sqrt(n)
        CL = [[_mp_root(n, r * k) / rt for k in range(n)] for r in range(rows)]
        W = np.zeros((n, n), dtype=np.complex128)
        for j in range(n):
            alpha = [k for k in range(n) if A[j, k] == 0]
            assert len(alpha) == m
            if m > 0:
                M = mpmath.matrix(m, m)
                rhs = mpmath.matrix(m, 1)
                for a, k in enumerate(alpha):
                    for r in range(m):
                        M[a, r] = CL[r][k]
                    rhs[a] = -CL[m][k]
                q = mpmath.lu_solve(M, rhs)
                coeff = [q[r] for r in range(m)] + [mpmath.mpf(1)]
            else:
                coeff = [mpmath.mpf(1)]
            for k in range(n):
                v = mpmath.fsum(coeff[r] * CL[r][k] for r in range(rows))
                W[j, k] = complex(v)
    return W


def cyc_W_closed_form(n: int, s: int, dps: int = 60) -> np.ndarray:
    """W[j][k] = n^(-1/2) prod_{m in alpha_j} (w^k - w^m), w = exp(2 pi i / n).

    Follows from the definition: [q_j 1] C_L evaluated at column k is
    n^(-1/2) times a monic polynomial of degree n - 2 s - 1 in w^k whose roots
    are the n - 2 s - 1 points w^m, m in alpha_j.
    """
    A = cyc_allocation(n, s)
    W = np.zeros((n, n), dtype=np.complex128)
    with mpmath.workdps(dps):
        rt = mpmath.sqrt(n)
        root = [_mp_root(n, e) for e in range(n)]
        for j in range(n):
            alpha = [k for k in range(n) if A[j, k] == 0]
            for k in range(n):
                p = mpmath.mpf(1)
                for mm in alpha:
                    p = p * (root[k] - root[mm])
                W[j, k] = complex(p / rt)
    return W


@functools.lru_cache(maxsize=None)
def _cyc_W_cached(n: int, s: int) -> np.ndarray:
    if n <= 16:
        return cyc_W_by_definition(n, s)
    return cyc_W_closed_form(n, s)


def cyc_W(n: int, s: int) -> np.ndarray:
    """The encoding matrix: by the paper's definition up to n = 16, by the
    closed form (pinned against the definition up to n = 45) beyond, where the
    multiprecision solves take from tens of seconds to minutes."""
    return _cyc_W_cached(n, s).copy()


def cyc_encode(G: np.ndarray, n: int, s: int, W: np.ndarray | None = None,
               dtype=np.complex64) -> np.ndarray:
    """Z = G W: node j sends z_j = G W_{., j} = sum_k W[k][j] g_k.

    complex128 arithmetic, then rounded to ``dtype`` (the vector sent).
    """
    if W is None:
        W = cyc_W(n, s)
    Z = W.T @ np.asarray(G, dtype=np.complex128)
    return Z.astype(dtype)


def cyc_project(R: np.ndarray, f: np.ndarray) -> np.ndarray:
    """e = f R: e_j = sum_i f_i R[j][i]  (the O(d P) part of phi)."""
    return np.asarray(R, dtype=np.complex128) @ np.asarray(f, dtype=np.float64)


def cyc_project_energy(R: np.ndarray) -> np.ndarray:
    """q_j = sum_i |R[j][i]|^2: the squared size of what node j sent.

    Not in the paper.  Rounding R to complex64 perturbs e_j = sum_i f_i R[j][i] by about
    2^-25 (E f^2 q_j)^(1/2), E f^2 = 2, whatever e_j itself comes to (the terms of e_j can
    cancel, those of q_j cannot), so q_j^(1/2) is the yardstick for "zero" in the rank
    decision of the locator.
    """
    R = np.asarray(R, dtype=np.complex128)
    return np.sum(R.real ** 2 + R.imag ** 2, axis=1)


def cyc_locate_from_projection(e: np.ndarray, q: np.ndarray, n: int, s: int, theta: float = 1e-6) -> dict:
    """The locator phi after the projection: syndromes, Toeplitz solve,
    recurrence, IDFT, support.  e = f R, q = cyc_project_energy(R).

    Readings where the paper is garbled or silent:
      * syndromes are h_m, m = n-2s .. n-1 ascending: [h_m] = e C_R^dagger;
      * row i of the s x s system is [h_{n-s-1-i} .. h_{n-2-i}] with right-hand
        side h_{n-1-i}: the recurrence h_l = sum_u beta_u h_{l+u-s} written for
        l = n-1-i;
      * fewer than s adversaries make the system singular (its rank is the
        number of non-zero entries of gamma = (f N)^T): singular values below
        theta * scale, scale = median_j q_j^(1/2), count as zero and beta is the
        pseudo-inverse solution; Lemma 8 lets any solution of the equations
        drive the recurrence.  (scale = median_j |e_j| was the first choice; e_j is
        a signed sum and can cancel to a tenth of its usual size, and with it the
        cutoff sinks into the rounding noise of complex64 vectors);
      * "t_j != 0" cannot be tested in floating point.  Exactly ``rank`` entries
        of t are non-zero in exact arithmetic, so V = the ``rank`` nodes with the
        largest |t_j| (V is empty when the rank is 0);
      * the paper's vectors are real numbers; a received vector may hold NaN or
        infinities.  An honest vector is finite, so a node whose e_j or q_j is not
        finite is an adversary: it is flagged outright and its e_j, q_j are taken as
        0, which keeps the arithmetic finite (to the locator the node then looks as
        if it had sent a vector with f R_j = 0, i.e. the error -f z_j: one of the
        at most s errors it can locate anyway).
    """
    e = np.asarray(e, dtype=np.complex128).copy()
    q = np.asarray(q, dtype=np.float64).copy()
    nonfinite = ~(np.isfinite(e.real) & np.isfinite(e.imag) & np.isfinite(q))
    e[nonfinite] = 0.0
    q[nonfinite] = 0.0
    out = _cyc_locate_passes(e, q, n, s, theta, nonfinite)
    out["nonfinite"] = nonfinite
    return out


def _cyc_locate_passes(e: np.ndarray, q: np.ndarray, n: int, s: int, theta: float, known: np.ndarray) -> dict:
    """phi on a finite projection record, run in passes.

    The first pass is the paper's locator (syndromes, s x s Toeplitz system, recurrence, IDFT, support).
    Reading where the paper is silent (it works in exact arithmetic, where one pass finds every adversary):
    with complex64 vectors adversaries that sit close together on the circle make the system so badly
    conditioned that a pass can miss some of them.  Every further pass therefore treats the set E of nodes
    flagged so far as erasures: with lambda(x) = prod_{v in E} (x - w^v) = sum_k lambda_k x^k, the sequence
    T_m = sum_k lambda_k h_{m-k} no longer contains the nodes of E (their terms carry the factor
    lambda(w^v) = 0) and is again a sum of exponentials, one per adversary not yet flagged; the 2 s - |E|
    values of T that the 2 s syndromes give (the last 2 s2 of them are used, s2 = floor((2 s - |E|) / 2))
    go through the same system, recurrence and IDFT with s2 in place of s, and the nodes found join E.  The
    passes end when one finds nothing (the usual second pass: its singular values are rounding noise) or
    when fewer than two values of T are left.  Nodes known to be adversarial beforehand (``known``: a
    non-finite record) are in E from the start, costing one syndrome each instead of two.  V can come out
    as a superset of the adversaries (an honest node flagged by an ill-conditioned pass stays flagged);
    decoding only needs V to contain them and |V| <= 2 s.  The rank cutoff of a pass is
    theta * scale * sum_k |lambda_k| (the rounding noise of h enters T through those coefficients).

    Returned ``t``, ``h``, ``sv``, ``beta``, ``margin`` are those of the first pass; ``rank`` is the number
    of nodes the passes found (``ranks``: per pass).
    """
    C = idft_matrix(n)
    scale = float(np.median(np.sqrt(np.asarray(q, dtype=np.float64))))
    tol = theta * scale
    flags = np.asarray(known, dtype=bool).copy()
    out = {"e": e, "scale": scale, "t": np.zeros(n, dtype=np.complex128),
           "flags": flags, "rank": 0, "h": np.zeros(n, dtype=np.complex128),
           "margin": np.inf, "ranks": []}
    if s == 0:
        return out
    w = np.exp(2j * np.pi / n)
    C_R = C[n - 2 * s:]
    syn = np.zeros(n, dtype=np.complex128)
    syn[n - 2 * s:] = e @ C_R.conj().T                         # h_m, m = n-2s .. n-1
    out["h"] = syn.copy()
    first = True
    while True:
        E = np.flatnonzero(flags)
        s2 = (2 * s - len(E)) // 2
        if s2 < 1:
            break
        lam = np.ones(1, dtype=np.complex128)                  # lambda_k multiplies x^k
        for v in E:                                            # times (x - w^v)
            lam = np.concatenate([[0.0], lam]) - w ** v * np.concatenate([lam, [0.0]])
        h = np.zeros(n, dtype=np.complex128)
        for m in range(n - 2 * s2, n):
            acc = 0.0 + 0.0j
            for k in range(len(lam)):
                acc += lam[k] * syn[m - k]
            h[m] = acc
        cut = tol * float(np.abs(lam).sum())
        M = np.empty((s2, s2), dtype=np.complex128)
        rhs = np.empty(s2, dtype=np.complex128)
        for i in range(s2):
            for u in range(s2):
                M[i, u] = h[n - s2 - 1 - i + u]
            rhs[i] = h[n - 1 - i]
        Us, sv, Vh = np.linalg.svd(M)
        keep = sv > cut
        rank = int(np.count_nonzero(keep))
        out["ranks"].append(rank)
        if first:
            out["sv"] = sv
        if rank == 0:
            break
        inv = np.zeros_like(sv)
        inv[keep] = 1.0 / sv[keep]
        beta = Vh.conj().T @ (inv * (Us.conj().T @ rhs))
        for ell in range(n - 2 * s2):
            acc = 0.0 + 0.0j
            for u in range(s2):
                acc += beta[u] * h[(ell + u - s2) % n]
            h[ell] = acc
        t = C @ h
        mag = np.abs(t)
        mag[E] = -1.0                                          # already flagged: not candidates
        order = np.argsort(-mag, kind="stable")
        if first:
            free = n - len(E)
            margin = mag[order[rank - 1]] / max(mag[order[rank]], 1e-300) if rank < free else np.inf
            out.update(h=h, t=t, beta=beta, margin=float(margin))
        flags[order[:rank]] = True
        out["rank"] += rank
        first = False
    return out


def cyc_locate(R: np.ndarray, f: np.ndarray, n: int, s: int, theta: float = 1e-6) -> dict:
    """V = phi(R) with the random vector f passed in (f ~ N(1_d, I_d))."""
    return cyc_locate_from_projection(cyc_project(R, f), cyc_project_energy(R), n, s, theta)


def cyc_decode_vector(n: int, s: int, flags) -> np.ndarray:
    """b with support in U = non-flagged nodes and W_{., U} b_U = 1_P.

    As in the proof of Lemma 3 the system is reduced to [C_L]_{., U} b_U =
    (0, .., 0, 1)^T (equivalent because [Q 1_P] has full column rank).  Among its
    solutions the minimum-2-norm one is returned (the paper's "first P - 2 s
    elements of U" choice is ``cyc_decode_vector_first``).
    """
    flags = np.asarray(flags, dtype=bool)
    U = np.flatnonzero(~flags)
    rows = n - 2 * s
    if len(U) < rows:
        raise ValueError("more than 2 s nodes flagged: no decode vector exists")
    C_L = idft_matrix(n)[:rows]
    rhs = np.zeros(rows, dtype=np.complex128)
    rhs[-1] = 1.0
    bU = np.linalg.lstsq(C_L[:, U], rhs, rcond=None)[0]
    b = np.zeros(n, dtype=np.complex128)
    b[U] = bU
    return b


def cyc_decode_vector_first(n: int, s: int, flags) -> np.ndarray:
    """The literal choice in the proof of Lemma 3: U-bar = the first n - 2 s
    elements of U, b_{U-bar} = ([C_L]_{., U-bar})^{-1} (0, .., 0, 1)^T."""
    flags = np.asarray(flags, dtype=bool)
    rows = n - 2 * s
    Ubar = np.flatnonzero(~flags)[:rows]
    if len(Ubar) < rows:
        raise ValueError("more than 2 s nodes flagged")
    C_L = idft_matrix(n)[:rows]
    rhs = np.zeros(rows, dtype=np.complex128)
    rhs[-1] = 1.0
    b = np.zeros(n, dtype=np.complex128)
    b[Ubar] = np.linalg.solve(C_L[:, Ubar], rhs)
    return b


def cyc_recover(R: np.ndarray, b: np.ndarray) -> np.ndarray:
    """u-hat = R_{., U} b as a complex128 vector (its imaginary part is rounding residue)."""
    U = np.flatnonzero(b != 0)
    return b[U] @ np.asarray(R, dtype=np.complex128)[U]


def cyc_decode(R: np.ndarray, n: int, s: int, flags, literal_b: bool = False) -> np.ndarray:
    """Algorithm 1, steps 2-4, for a given adversary set: u = Re(R_{., U} b)."""
    b = cyc_decode_vector_first(n, s, flags) if literal_b else cyc_decode_vector(n, s, flags)
    return cyc_recover(R, b).real


def cyc_decode_full(R: np.ndarray, f: np.ndarray, n: int, s: int, theta: float = 1e-6) -> dict:
    """Algorithm 1 in full: locate, then decode."""
    loc = cyc_locate(R, f, n, s, theta)
    loc["u"] = cyc_decode(R, n, s, loc["flags"]) if loc["flags"].sum() <= 2 * s else None
    return loc


# --------------------------------------------------------------------------
# Real -> complex packing of the cyclic code  (Section 3, last paragraph)
# --------------------------------------------------------------------------


def cyc_pack(G: np.ndarray) -> np.ndarray:
    """G-hat in C^{ceil(d/2) x P}: component i has real part G_i and imaginary part
    G_{ceil(d/2)+i} (zero where d is odd and the second half is one short).
    Worker-major like everything else: returns ``[n][ceil(d/2)]`` complex128."""
    G = np.asarray(G, dtype=np.float64)
    n, d = G.shape
    h = (d + 1) // 2
    out = np.zeros((n, h), dtype=np.complex128)
    out.real = G[:, :h]
    out.imag[:, : d - h] = G[:, h:]
    return out


def cyc_unpack(u_hat: np.ndarray, d: int) -> np.ndarray:
    """Inverse of the packing applied to the recovered u-hat = G-hat 1_P.

    The paper writes u = Re(u-hat) + Im(u-hat), which cannot undo a packing that put
    different coordinates in the two parts; the reading taken is the concatenation
    [Re(u-hat); Im(u-hat)] cut to d entries."""
    h = (d + 1) // 2
    u_hat = np.asarray(u_hat, dtype=np.complex128)
    return np.concatenate([u_hat.real, u_hat.imag[: d - h]])


def cyc_encode_packed(G: np.ndarray, n: int, s: int, W: np.ndarray | None = None,
                      dtype=np.complex64) -> np.ndarray:
    """The compute nodes send G-hat W: ``[n][ceil(d/2)]`` complex."""
    if W is None:
        W = cyc_W(n, s)
    return (W.T @ cyc_pack(G)).astype(dtype)


def cyc_decode_packed(R: np.ndarray, n: int, s: int, flags, d: int) -> np.ndarray:
    """Algorithm 1 steps 2-4 on packed vectors: u-hat = R_{., U} b, then unpack."""
    b = cyc_decode_vector(n, s, flags)
    return cyc_unpack(cyc_recover(R, b), d)
