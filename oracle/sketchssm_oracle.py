"""CPU oracle for the SketchSSM decode path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, float64 NumPy statement of what the decode hot path computes:
the token-by-token recurrences of Mamba-2 (scalar decay, no erase), GDN (gated
delta rule, scalar decay) and KDA (delta rule, per-channel decay); the periodic
state update that replays the buffered tokens and refreshes the sketch; the
per-token decode step that reads only the sketch; the exact full-state-read
decode; and the offline fit of the sketching matrix and the fixed coefficient
map.  Nothing here is blocked, fused or reordered beyond what the paper's
definitions state.  It shares no code with the CUDA library and must never be
imported by it: only the tests, the smoke check and the benchmark's CPU-baseline
leg call it.  All inputs are NumPy arrays (any float dtype, widened to float64).

Notation (paper -> here): K = key/query channels, V = value channels,
G = sketch rank r, W = window length L, S_0 in R^{K x V} the state at the start
of the window, Omega in R^{K x G}, sketch U = S_0^T Omega in R^{V x G},
coefficient map C in R^{G x K}.

Every function broadcasts over leading "head" axes: a state is [..., K, V],
a key [..., K], a scalar gate [...].

A *token* is the tuple (k, v, beta, decay): decay is the scalar a_t (Mamba-2),
the scalar alpha_t (GDN) or the vector g_t in (0,1)^K (KDA).

Pinned by tests/test_oracle_pins.py against: the exact decomposition of the
read (Eq. 4), explicit dense transition matrices built with Python loops, the
identity-basis special case, replay == repeated single updates, the empty-buffer
case, the WY identities (Eq. 41-45; the projected erase vectors against C times
the erase factors), the PCA closed forms of Appendix A.1, the
traffic-reduction values printed in Tables 4-7, and for the state-dependent
coefficient maps of Appendix A.2: a library least-squares solve of the ridge
problem, the range projection in the limit of no ridge, independence of the
orthogonal completion, the Woodbury step against a dense inverse, exactness of
the pivot approximation when P >= G, a hand-rolled brute force on tiny heads, and the sketch-form restatements
(*_from_sketch) against the appendix forms at the exact sketch.  Absolute output values on
the benchmark workloads have no printed counterpart in the paper: for those,
parity is pinned only through the identities above ("parity unpinned" by a
worked numeric example).
"""
from __future__ import annotations

import numpy as np

MAMBA2, GDN, KDA = "mamba2", "gdn", "kda"
_KINDS = (MAMBA2, GDN, KDA)


def _f64(x):
    return np.asarray(x, dtype=np.float64)


def _decay_diag(kind, decay, K):
    """diag(D_t) as an array [..., K] (Section 3.1: D_t is the decay matrix)."""
    d = _f64(decay)
    if kind == KDA:
        assert d.shape[-1] == K
        return d
    return np.broadcast_to(d[..., None], d.shape + (K,))


# ----------------------------------------------------------------------------
# Recurrence (Section 3.1, Eq. 1 and Eq. 3)
# ----------------------------------------------------------------------------

def transition(kind, S, k, v, beta, decay):
    """One token of the recurrence, S_t from S_{t-1}.

    Eq. (1): S_t = D_t S_{t-1} + k_t w_t^T with the write vector
    w_t = beta_t (v_t - S_{t-1}^T D_t^T k_t) for the delta-rule models (GDN, KDA)
    and w_t = beta_t v_t for Mamba-2 (M_t = D_t, no erase).  This is the same
    map as Eq. (3), S_t = M_t S_{t-1} + beta_t k_t v_t^T with
    M_t = (I - beta_t k_t k_t^T) D_t: decay first, then erase.
    """
    assert kind in _KINDS
    S, k, v, beta = _f64(S), _f64(k), _f64(v), _f64(beta)
    K = S.shape[-2]
    d = _decay_diag(kind, decay, K)
    DS = d[..., :, None] * S                                  # D_t S_{t-1}
    if kind == MAMBA2:
        w = beta[..., None] * v
    else:
        erase = np.einsum("...kv,...k->...v", DS, k)          # (D_t S_{t-1})^T k_t = S_{t-1}^T D_t^T k_t
        w = beta[..., None] * (v - erase)
    return DS + k[..., :, None] * w[..., None, :]


def exact_read(S, q):
    """o_t = S_t^T q_t (Eq. 2 / Eq. 4, left-hand side)."""
    return np.einsum("...kv,...k->...v", _f64(S), _f64(q))


def sketch_of(S, Omega):
    """U = S^T Omega in R^{V x G} (Eq. 7)."""
    return np.einsum("...kv,...kg->...vg", _f64(S), _f64(Omega))


def round_bf16(x):
    """Round to the nearest bfloat16 (ties to even), returned as float64: the storage precision the paper uses for the
    sketch, the coefficient map and the erase vectors (Appendix D, Appendix F setup).  The value is first rounded to
    float32, the precision the sketch is formed in before it is stored."""
    bits = np.ascontiguousarray(_f64(x).astype(np.float32)).view(np.uint32).astype(np.uint64)
    rounded = ((bits + 0x7FFF + ((bits >> 16) & 1)) >> 16) << 16
    return rounded.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(x))


# ----------------------------------------------------------------------------
# Read decomposition (Section 3.1, Eq. 4)
# ----------------------------------------------------------------------------

def effective_query(kind, tokens, q):
    """Effective query and buffer weights of Eq. (4) by their definitions.

    q~_t = M_{1:t}^T q_t = M_1^T M_2^T ... M_t^T q_t with
    M_s^T = D_s (I - beta_s k_s k_s^T) (Mamba-2: M_s^T = D_s), applied from
    s = t down to s = 1.  Before M_s^T is applied the running vector equals
    M_{s+1:t}^T q_t, so a_s = beta_s <k_s, M_{s+1:t}^T q_t>
    = beta_s <M_{s+1:t} k_s, q_t> is the weight of v_s in o_t^buffer.

    tokens: list of (k, v, beta, decay) in arrival order, the last one being the
    current token t.  Returns (q~_t [..., K], [a_1..a_t] each [...]).
    """
    x = _f64(q).copy()
    K = x.shape[-1]
    a = [None] * len(tokens)
    for s in range(len(tokens) - 1, -1, -1):
        k, _v, beta, decay = tokens[s]
        k, beta = _f64(k), _f64(beta)
        a[s] = beta * np.einsum("...k,...k->...", k, x)
        if kind != MAMBA2:
            x = x - k * a[s][..., None]                       # (I - beta_s k_s k_s^T) x
        x = _decay_diag(kind, decay, K) * x                   # D_s (.)
    return x, a


def buffer_output(tokens, a):
    """o_t^buffer = sum_s a_s v_s (Eq. 4)."""
    out = 0.0
    for (_k, v, _b, _d), a_s in zip(tokens, a):
        out = out + a_s[..., None] * _f64(v)
    return out


def full_read_decode(kind, S0, tokens, q):
    """Exact decode output from the window-start state: S_0^T q~_t + o_t^buffer (Eq. 4)."""
    x, a = effective_query(kind, tokens, q)
    V = _f64(S0).shape[-1]
    ob = buffer_output(tokens, a) if tokens else np.zeros(x.shape[:-1] + (V,))
    return exact_read(S0, x) + ob


def decode_step(kind, U, C, tokens, q, erase_store=None):
    """Non-flush decode step of Algorithm 1: o_t = U C q~_t + o_t^buffer.

    U [..., V, G] is the sketch of the window-start state, C [..., G, K] the
    coefficient map; c_t = C q~_t (Section 4.1, "Per-step: coefficient vector").
    `tokens` already contains the current token (Algorithm 1 appends first).
    erase_store: if given (GDN / KDA), c_t is formed from projected erase vectors (Eq. 44-45) each of which is passed
    through this function when it is stored (e.g. round_bf16: the paper keeps the vectors in BF16); with the identity
    this is the same c_t.
    """
    x, a = effective_query(kind, tokens, q)
    if erase_store is None:
        c = np.einsum("...gk,...k->...g", _f64(C), x)
    else:
        c = wy_coefficients(kind, tokens, q, C, store=erase_store)
    o_state = np.einsum("...vg,...g->...v", _f64(U), c)
    ob = buffer_output(tokens, a) if tokens else 0.0
    return o_state + ob


def state_update(kind, S0, tokens, Omega, q=None):
    """Flush step of Algorithm 1: replay the buffered tokens exactly, then
    o = S^T q from the updated state (if q is given) and U = S^T Omega.

    Returns (S_new, U, o or None)."""
    S = _f64(S0)
    for (k, v, beta, decay) in tokens:
        S = transition(kind, S, k, v, beta, decay)
    o = exact_read(S, q) if q is not None else None
    return S, sketch_of(S, Omega), o


def run_schedule(kind, S_init, Omega, C, step_tokens, step_queries, L):
    """Algorithm 1, inference part, for len(step_tokens) decode steps.

    Initial sketch from S_init; then windows of L steps: L-1 non-flush decode
    steps followed by one flush step whose output is exact.  Returns
    (outputs list, S, U, tokens still buffered).
    """
    S = _f64(S_init)
    U = sketch_of(S, Omega)
    ring, outs = [], []
    for tok, q in zip(step_tokens, step_queries):
        ring.append(tok)
        if len(ring) < L:
            outs.append(decode_step(kind, U, C, ring, q))
        else:
            S, U, o = state_update(kind, S, ring, Omega, q)
            outs.append(o)
            ring = []
    return outs, S, U, ring


# ----------------------------------------------------------------------------
# WY form of the transition product (Appendix C, Eq. 38-45)
# ----------------------------------------------------------------------------

def wy_factors(kind, tokens):
    """Erase factors pi_s and cumulative diagonals d_[s] of Eq. (41)-(42).

    d_[s] = diag(D_s ... D_1); l_j(s) = (D_s ... D_{j+1}) k_j (Eq. 40), formed
    as a running product (never as a quotient of cumulative diagonals);
    pi_s = beta_s (d_[s] * k_s - sum_{j<s} <l_j(s), k_s> pi_j), pi_1 = beta_1 d_[1] * k_1.
    Returns (d list, pi list, l list) where l[j] = l_j(t) for t = len(tokens).
    """
    assert kind != MAMBA2
    K = _f64(tokens[0][0]).shape[-1]
    d_cum, pis, ls = [], [], []
    d_run = None
    for s, (k, _v, beta, decay) in enumerate(tokens):
        k, beta = _f64(k), _f64(beta)
        Ds = _decay_diag(kind, decay, K)
        d_run = Ds.copy() if d_run is None else Ds * d_run
        ls = [Ds * l for l in ls]                              # l_j(s) = D_s l_j(s-1)
        acc = d_run * k
        for l_j, pi_j in zip(ls, pis):
            acc = acc - np.einsum("...k,...k->...", l_j, k)[..., None] * pi_j
        pis.append(beta[..., None] * acc)
        ls.append(k.copy())                                    # l_s(s) = k_s (empty product)
        d_cum.append(d_run.copy())
    return d_cum, pis, ls


def wy_effective_query(kind, tokens, q):
    """q~_t = d_[t] * q_t - sum_s pi_s <l_s(t), q_t> (Eq. 43); Mamba-2: d_[t] * q_t."""
    q = _f64(q)
    K = q.shape[-1]
    if kind == MAMBA2:
        d = np.ones_like(q)
        for (_k, _v, _b, decay) in tokens:
            d = _decay_diag(kind, decay, K) * d
        return d * q
    d_cum, pis, ls = wy_factors(kind, tokens)
    out = d_cum[-1] * q
    for l_s, pi_s in zip(ls, pis):
        out = out - pi_s * np.einsum("...k,...k->...", l_s, q)[..., None]
    return out


def projected_erase_vectors(kind, tokens, C, store=None):
    """f_s = beta_s [C (d_[s] * k_s) - sum_{j<s} f_j <l_j(s), k_s>] for every buffered token (Eq. 45),
    with the left factors l_j(s) = (D_s ... D_{j+1}) k_j kept as running products.
    store: applied to every f_s when it is stored (default: nothing); later vectors are formed from the stored ones.
    Returns (f list, l list, d) where l[j] = l_j(t) and d = d_[t] for t = len(tokens)."""
    assert kind != MAMBA2
    C = _f64(C)
    K = C.shape[-1]
    fs, ls = [], []
    d_run = None
    for (k, _v, beta, decay) in tokens:
        k, beta = _f64(k), _f64(beta)
        Ds = _decay_diag(kind, decay, K)
        d_run = Ds.copy() if d_run is None else Ds * d_run
        ls = [Ds * l for l in ls]
        acc = np.einsum("...gk,...k->...g", C, d_run * k)
        for l_j, f_j in zip(ls, fs):
            acc = acc - f_j * np.einsum("...k,...k->...", l_j, k)[..., None]
        f_s = beta[..., None] * acc
        fs.append(f_s if store is None else _f64(store(f_s)))
        ls.append(k.copy())
    return fs, ls, d_run


def wy_coefficients(kind, tokens, q, C, store=None):
    """c_t = C (d_[t] * q_t) - sum_s f_s <l_s(t), q_t> with the projected erase
    factors f_s of Eq. 45 (Eq. 44), each passed through `store` when it is stored."""
    q, C = _f64(q), _f64(C)
    fs, ls, d_run = projected_erase_vectors(kind, tokens, C, store)
    c = np.einsum("...gk,...k->...g", C, d_run * q)
    for l_s, f_s in zip(ls, fs):
        c = c - f_s * np.einsum("...k,...k->...", l_s, q)[..., None]
    return c


# ----------------------------------------------------------------------------
# Offline calibration (Section 4.1, Eq. 8 and Eq. 10; Appendix A.1)
# ----------------------------------------------------------------------------

def _sym_powers(E0, rcond=1e-12):
    """E0^{1/2} and the Moore-Penrose E0^{-1/2} on the support of E0 (end of Appendix A.1)."""
    lam, P = np.linalg.eigh(_f64(E0))
    keep = lam > rcond * lam.max()
    root = np.where(keep, np.sqrt(np.where(keep, lam, 1.0)), 0.0)
    iroot = np.where(keep, 1.0 / np.where(keep, root, 1.0), 0.0)
    return (P * root) @ P.T, (P * iroot) @ P.T


def fit_sketching_matrix(Qt, E0, G):
    """Uncentered PCA of the state-weighted queries (Appendix A.1, Steps 1-5).

    z_i = E0^{1/2} q~_i; C_z = mean z z^T; P_G = eigenvectors of the G largest
    eigenvalues; Omega* = E0^{-1/2} P_G.  Eigenvectors are ordered by decreasing
    eigenvalue and signed so that their largest-magnitude entry is positive.
    Returns (Omega [K, G], eigenvalues [K] descending).
    """
    Qt = _f64(Qt)
    E_half, E_ihalf = _sym_powers(E0)
    Z = Qt @ E_half                                           # rows z_i^T (E_half symmetric)
    Cz = Z.T @ Z / Z.shape[0]
    lam, P = np.linalg.eigh(Cz)
    order = np.argsort(-lam, kind="stable")
    lam, P = lam[order], P[:, order]
    sign = np.sign(P[np.abs(P).argmax(axis=0), np.arange(P.shape[1])])
    P = P * np.where(sign == 0, 1.0, sign)[None, :]
    return E_ihalf @ P[:, :G], lam


def offline_coefficient_map(Omega, E0):
    """C_offline = (Omega^T E0 Omega)^+ Omega^T E0 (Eq. 10)."""
    Omega, E0 = _f64(Omega), _f64(E0)
    return np.linalg.pinv(Omega.T @ E0 @ Omega) @ Omega.T @ E0


def state_dependent_coefficient_map(S0, U):
    """C = (U^T U)^+ U^T S_0^T (Eq. 9), the least-squares map for the current state."""
    S0, U = _f64(S0), _f64(U)
    return np.linalg.pinv(U.T @ U) @ U.T @ S0.T


def _orthogonal_completion(Omega):
    """R in R^{K x K} with R^T R = I whose first G rows are Omega^T (Appendix A.2.2, Step 1: the orthonormal
    sketching matrix completed to an orthogonal matrix R^T = [Omega | Omega_perp], so that Omega = R^T J)."""
    Omega = _f64(Omega)
    K, G = Omega.shape
    assert np.allclose(Omega.T @ Omega, np.eye(G), atol=1e-5), "Appendix A.2.2 assumes an orthonormal sketching matrix"
    Uf, _s, _vt = np.linalg.svd(Omega, full_matrices=True)        # columns G.. of Uf span the complement of range(Omega)
    return np.concatenate([Omega, Uf[:, G:]], axis=1).T


def _rotated_metric(S0, Omega):
    """S'_0 = R S_0, x-coordinates R, the normalisation mu = ||S'_0||_F^2 / K (mu = 1 for a zero state) and the
    normalised state metric H = S'_0 S'_0^T / mu (Eq. 26-27)."""
    S0 = _f64(S0)
    K = S0.shape[0]
    R = _orthogonal_completion(Omega)
    Sp = R @ S0
    mu = float(np.sum(Sp * Sp)) / K
    if mu == 0.0:
        mu = 1.0
    return R, Sp, mu, Sp @ Sp.T / mu


def ridge_coefficient_map(S0, Omega, lam=0.1):
    """Exact regularised state-dependent coefficient map of one head (Appendix A.2.2, Step 1, Eq. 28-29).

    In the basis-aligned coordinates x_t = R q~_t the coefficient vector minimises
    (x_t - J c)^T H (x_t - J c) + lam ||c||^2, so c = (J^T H J + lam I_G)^{-1} J^T H x_t with J the first G
    coordinate vectors.  Returned as the map C [G, K] acting on the effective query itself: c = C q~_t.
    S0 [K, V], Omega [K, G] orthonormal.
    """
    Omega = _f64(Omega)
    K, G = Omega.shape
    R, _Sp, _mu, H = _rotated_metric(S0, Omega)
    J = np.eye(K)[:, :G]
    return np.linalg.solve(J.T @ H @ J + lam * np.eye(G), J.T @ H) @ R


def pivot_metric_factors(S0, Omega, P=4):
    """The low-rank-plus-diagonal factors of Appendix A.2.2, Step 2 (Eq. 30-33), for one head.

    p = min(G, P); Q [V, p] is an orthonormal basis of the first p columns of the sketch U = S'_0^T J, built by
    Gram-Schmidt in column order (a column that lies in the span of its predecessors contributes a zero column);
    L = S'_0 Q / sqrt(mu) [K, p]; d_i = max(H_ii - ||L_i||^2, 0).  Returns (R, mu, Q, L, d).
    """
    Omega = _f64(Omega)
    K, G = Omega.shape
    R, Sp, mu, H = _rotated_metric(S0, Omega)
    p = min(G, P)
    J = np.eye(K)[:, :G]
    U = Sp.T @ J                                                   # the current sketch, V x G
    Q = np.zeros((U.shape[0], p))
    for j in range(p):
        u = U[:, j].copy()
        for i in range(j):
            u -= Q[:, i] * (Q[:, i] @ U[:, j])
        for i in range(j):                                         # second sweep: re-orthogonalise
            u -= Q[:, i] * (Q[:, i] @ u)
        nrm, ref = np.linalg.norm(u), np.linalg.norm(U[:, j])
        Q[:, j] = u / nrm if nrm > 1e-10 * max(ref, 1e-300) and ref > 0 else 0.0
    L = Sp @ Q / np.sqrt(mu)
    d = np.maximum(np.diag(H) - np.sum(L * L, axis=1), 0.0)
    return R, mu, Q, L, d


def pivot_coefficient_map(S0, Omega, lam=0.1, P=4):
    """State-dependent coefficient map with the approximated state metric H^ = L L^T + Diag(d)
    (Appendix A.2.2, Steps 2-4, Eq. 30-37), for one head; returns C [G, K] with c_t = C q~_t.

    With L_G = J^T L, D_G = Diag(J^T d) + lam I:  c = (D_G + L_G L_G^T)^{-1} [L_G (L^T x_t) + J^T Diag(d) x_t],
    the inverse taken through the Woodbury identity with the p x p system T_P = I_p + L_G^T D_G^{-1} L_G.
    """
    Omega = _f64(Omega)
    K, G = Omega.shape
    R, _mu, _Q, L, d = pivot_metric_factors(S0, Omega, P)
    p = L.shape[1]
    J = np.eye(K)[:, :G]
    LG = J.T @ L                                                   # G x p
    DG = J.T @ d + lam                                             # diagonal of D_G
    rhs = LG @ L.T + J.T @ np.diag(d)                              # G x K: maps x_t to J^T H^ x_t
    TP = np.eye(p) + LG.T @ (LG / DG[:, None])
    Dinv_rhs = rhs / DG[:, None]
    A_inv_rhs = Dinv_rhs - (LG / DG[:, None]) @ np.linalg.solve(TP, LG.T @ Dinv_rhs)
    return A_inv_rhs @ R


def ridge_coefficient_map_from_sketch(S0, U, lam=0.1):
    """The ridge map of Eq. 28-29 carried back from the rotated coordinates to the quantities a kernel holds
    (J^T H J = U^T U / mu, J^T H R = U^T S_0^T / mu for U = S_0^T Omega):  C = (U^T U + lam mu I)^{-1} U^T S_0^T,
    mu = ||S_0||_F^2 / K (1 for a zero state).  Equal to ridge_coefficient_map when U is the exact sketch; stated in
    terms of U so that it also defines the map built from a sketch that was rounded when it was stored.
    S0 [K, V], U [V, G]."""
    S0, U = _f64(S0), _f64(U)
    K, G = S0.shape[0], U.shape[1]
    mu = float(np.sum(S0 * S0)) / K
    if mu == 0.0:
        mu = 1.0
    return np.linalg.solve(U.T @ U + lam * mu * np.eye(G), U.T @ S0.T)


def pivot_coefficient_map_from_sketch(S0, U, Omega, lam=0.1, P=4):
    """The approximated map of Eq. 30-37 in the same carried-back form: with Q the Gram-Schmidt basis of the first p
    sketch columns, L_G = U^T Q / sqrt(mu), d_g = max((||U_g||^2 - ||Q^T U_g||^2) / mu, 0), D_G = Diag(d) + lam I,
    C = (D_G + L_G L_G^T)^{-1} [L_G Q^T S_0^T / sqrt(mu) + Diag(d) Omega^T], the inverse through the p x p Woodbury
    system.  Equal to pivot_coefficient_map when U is the exact sketch.  S0 [K, V], U [V, G], Omega [K, G]."""
    S0, U, Omega = _f64(S0), _f64(U), _f64(Omega)
    K, G = Omega.shape
    mu = float(np.sum(S0 * S0)) / K
    if mu == 0.0:
        mu = 1.0
    p = min(G, P)
    Q = np.zeros((U.shape[0], p))
    for j in range(p):
        u = U[:, j].copy()
        for i in range(j):
            u -= Q[:, i] * (Q[:, i] @ U[:, j])
        for i in range(j):
            u -= Q[:, i] * (Q[:, i] @ u)
        nrm, ref = np.linalg.norm(u), np.linalg.norm(U[:, j])
        Q[:, j] = u / nrm if nrm > 1e-10 * max(ref, 1e-300) and ref > 0 else 0.0
    LG = U.T @ Q / np.sqrt(mu)                                     # G x p
    d = np.maximum((np.sum(U * U, axis=0) - np.sum((Q.T @ U) ** 2, axis=0)) / mu, 0.0)
    DG = d + lam
    rhs = LG @ (Q.T @ S0.T) / np.sqrt(mu) + d[:, None] * Omega.T   # G x K
    TP = np.eye(p) + LG.T @ (LG / DG[:, None])
    Dinv_rhs = rhs / DG[:, None]
    return Dinv_rhs - (LG / DG[:, None]) @ np.linalg.solve(TP, LG.T @ Dinv_rhs)


def coefficient_maps(S, Omega, mode, lam=0.1, P=4, U=None):
    """Per-head state-dependent maps for a batch of heads: S [N, K, V], Omega [N, K, G] -> C [N, G, K].
    mode "ridge": ridge_coefficient_map; mode "pivot": pivot_coefficient_map.  With U [N, V, G] given (the sketch as it
    was stored, e.g. rounded to bfloat16) the maps are built from that sketch by the *_from_sketch forms."""
    S, Omega = _f64(S), _f64(Omega)
    if U is not None:
        U = _f64(U)
        fn = {"ridge": lambda i: ridge_coefficient_map_from_sketch(S[i], U[i], lam),
              "pivot": lambda i: pivot_coefficient_map_from_sketch(S[i], U[i], Omega[i], lam, P)}[mode]
        return np.stack([fn(i) for i in range(S.shape[0])])
    fn = {"ridge": lambda s, o: ridge_coefficient_map(s, o, lam), "pivot": lambda s, o: pivot_coefficient_map(s, o, lam, P)}[mode]
    return np.stack([fn(S[i], Omega[i]) for i in range(S.shape[0])])


def run_schedule_state_dependent(kind, S_init, Omega, step_tokens, step_queries, L, mode, lam=0.1, P=4):
    """Algorithm 1 with the coefficient map rebuilt from the state at every flush (and from the initial state):
    "construct the initial U, C from S_0", then per window L-1 sketch reads and one exact flush followed by U, C.
    Heads on the leading axis: S_init [N, K, V], Omega [N, K, G].  Returns (outputs, S, U, C)."""
    S = _f64(S_init)
    U = sketch_of(S, Omega)
    C = coefficient_maps(S, Omega, mode, lam, P)
    ring, outs = [], []
    for tok, q in zip(step_tokens, step_queries):
        ring.append(tok)
        if len(ring) < L:
            outs.append(decode_step(kind, U, C, ring, q))
        else:
            S, U, o = state_update(kind, S, ring, Omega, q)
            C = coefficient_maps(S, Omega, mode, lam, P)
            outs.append(o)
            ring = []
    return outs, S, U, C


# ----------------------------------------------------------------------------
# Traffic model (Appendix D, Table 3)
# ----------------------------------------------------------------------------

def nonflush_read_bytes(K, V, G, W, erase):
    """T_G = 2 G (V + K + e W): BF16 sketch, coefficient map and projected erase vectors."""
    return 2 * G * (V + K + (W if erase else 0))


def traffic_reduction(K, V, G, W, erase):
    """R_G = 8KV / ((W-1) T_G / W + 8KV / W): state traffic of Standard over SketchSSM."""
    return 8.0 * K * V / ((W - 1) * nonflush_read_bytes(K, V, G, W, erase) / W + 8.0 * K * V / W)


def replay_traffic_reduction(W):
    """ReplaySSM: 2D / (D + D/W) = 2W / (W + 1)."""
    return 2.0 * W / (W + 1.0)
