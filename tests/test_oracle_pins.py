"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests re-types an oracle formula: each compares the oracle with
an independent statement of the same quantity -- explicit dense transition
matrices multiplied with hand-written Python loops, a closed form, a special
case that collapses to a textbook routine, or a number printed in the paper.
"""
import itertools
import os
import random

import numpy as np
import pytest

from oracle import sketchssm_oracle as orc

KINDS = ("mamba2", "gdn", "kda")
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------------------
# helpers: random heads, and a brute-force model made of Python lists only
# ---------------------------------------------------------------------------

def rand_tokens(rng, kind, n, K, V, lead=()):
    toks = []
    for _ in range(n):
        k = rng.standard_normal(lead + (K,))
        if kind != "mamba2":
            k /= np.linalg.norm(k, axis=-1, keepdims=True)
        v = rng.standard_normal(lead + (V,))
        beta = rng.uniform(0.1, 0.95, lead)
        decay = rng.uniform(0.3, 0.99, lead + ((K,) if kind == "kda" else ()))
        toks.append((k, v, beta, decay))
    return toks


def mat_mul(A, B):
    n, m, p = len(A), len(B), len(B[0])
    return [[sum(A[i][l] * B[l][j] for l in range(m)) for j in range(p)] for i in range(n)]


def mat_T(A):
    return [list(r) for r in zip(*A)]


def dense_M(kind, k, beta, decay, K):
    """M_t = (I - beta k k^T) D_t as a K x K list of lists (Mamba-2: D_t)."""
    d = [float(decay[i]) if kind == "kda" else float(decay) for i in range(K)]
    D = [[d[i] if i == j else 0.0 for j in range(K)] for i in range(K)]
    if kind == "mamba2":
        return D
    E = [[(1.0 if i == j else 0.0) - float(beta) * float(k[i]) * float(k[j]) for j in range(K)] for i in range(K)]
    return mat_mul(E, D)


def brute_states(kind, S0, toks):
    """S_1..S_t by Eq. (3) with dense matrices: S_t = M_t S_{t-1} + beta_t k_t v_t^T."""
    K, V = len(S0), len(S0[0])
    S = [list(map(float, r)) for r in S0]
    out = []
    for (k, v, beta, decay) in toks:
        M = dense_M(kind, k, beta, decay, K)
        MS = mat_mul(M, S)
        S = [[MS[i][j] + float(beta) * float(k[i]) * float(v[j]) for j in range(V)] for i in range(K)]
        out.append(S)
    return out


def brute_prod(kind, toks, a, b, K):
    """M_{a:b} = M_b ... M_a (1-based, inclusive); identity if a > b."""
    P = [[1.0 if i == j else 0.0 for j in range(K)] for i in range(K)]
    for s in range(a, b + 1):
        k, _v, beta, decay = toks[s - 1]
        P = mat_mul(dense_M(kind, k, beta, decay, K), P)
    return P


# ---------------------------------------------------------------------------
# P5 / P8: brute force on tiny heads; D-form == M-form
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("K,V,n", [(3, 2, 3), (4, 4, 2), (2, 3, 1)])
def test_transition_matches_dense_matrix_recurrence(kind, K, V, n):
    rng = np.random.default_rng(100 + K * 7 + V + n)
    toks = rand_tokens(rng, kind, n, K, V)
    S0 = rng.standard_normal((K, V))
    ref = brute_states(kind, S0.tolist(), toks)
    S = S0
    for t, tok in enumerate(toks):
        S = orc.transition(kind, S, *tok)
        np.testing.assert_allclose(S, np.array(ref[t]), rtol=0, atol=1e-13)


@pytest.mark.parametrize("kind", KINDS)
def test_closed_form_of_the_update_eq3(kind):
    """S_t = M_{1:t} S_0 + sum_s beta_s (M_{s+1:t} k_s) v_s^T with explicit products."""
    K, V, n = 4, 3, 3
    rng = np.random.default_rng(7)
    toks = rand_tokens(rng, kind, n, K, V)
    S0 = rng.standard_normal((K, V))
    S, _U, _o = orc.state_update(kind, S0, toks, np.eye(K))
    ref = np.array(mat_mul(brute_prod(kind, toks, 1, n, K), S0.tolist()))
    for s in range(1, n + 1):
        k, v, beta, _ = toks[s - 1]
        Mk = np.array(brute_prod(kind, toks, s + 1, n, K)) @ k
        ref = ref + beta * np.outer(Mk, v)
    np.testing.assert_allclose(S, ref, rtol=0, atol=1e-13)


@pytest.mark.parametrize("kind", KINDS)
def test_effective_query_and_buffer_weights_brute_force(kind):
    """q~_t = M_{1:t}^T q_t and a_s = beta_s <M_{s+1:t} k_s, q_t> from dense products."""
    K, V, n = 4, 2, 3
    rng = np.random.default_rng(11)
    toks = rand_tokens(rng, kind, n, K, V)
    q = rng.standard_normal(K)
    x, a = orc.effective_query(kind, toks, q)
    M1t = brute_prod(kind, toks, 1, n, K)
    ref_x = [sum(M1t[i][j] * q[i] for i in range(K)) for j in range(K)]       # M^T q
    np.testing.assert_allclose(x, ref_x, rtol=0, atol=1e-13)
    for s in range(1, n + 1):
        k, _v, beta, _d = toks[s - 1]
        Ms = brute_prod(kind, toks, s + 1, n, K)
        Mk = [sum(Ms[i][j] * k[j] for j in range(K)) for i in range(K)]
        ref_a = beta * sum(Mk[i] * q[i] for i in range(K))
        assert abs(a[s - 1] - ref_a) < 1e-13


# ---------------------------------------------------------------------------
# P1: decomposition of the read (Eq. 4)
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("kind", KINDS)
def test_full_read_decode_equals_token_by_token_output(kind):
    K, V, n = 16, 12, 9
    rng = np.random.default_rng(3)
    lead = (2, 3)
    toks = rand_tokens(rng, kind, n, K, V, lead)
    S0 = rng.standard_normal(lead + (K, V))
    S = S0
    for t in range(n):
        S = orc.transition(kind, S, *toks[t])
        q = rng.standard_normal(lead + (K,))
        exact = orc.exact_read(S, q)
        got = orc.full_read_decode(kind, S0, toks[: t + 1], q)
        np.testing.assert_allclose(got, exact, rtol=0, atol=1e-11)


# ---------------------------------------------------------------------------
# P2: identity basis => sketch read is the exact read
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("kind", KINDS)
def test_identity_basis_makes_decode_step_exact(kind):
    K, V, n = 8, 5, 4
    rng = np.random.default_rng(5)
    toks = rand_tokens(rng, kind, n, K, V)
    S0 = rng.standard_normal((K, V))
    U = orc.sketch_of(S0, np.eye(K))
    np.testing.assert_array_equal(U, S0.T)
    S = S0
    for t in range(n):
        S = orc.transition(kind, S, *toks[t])
        q = rng.standard_normal(K)
        got = orc.decode_step(kind, U, np.eye(K), toks[: t + 1], q)
        np.testing.assert_allclose(got, S.T @ q, rtol=0, atol=1e-12)


def test_low_rank_basis_is_an_approximation_not_exact():
    """Guard against an oracle that ignores the sketch: with r < K the result must differ."""
    K, V = 8, 5
    rng = np.random.default_rng(6)
    toks = rand_tokens(rng, "gdn", 2, K, V)
    S0 = rng.standard_normal((K, V))
    Om = np.linalg.qr(rng.standard_normal((K, 3)))[0]
    q = rng.standard_normal(K)
    approx = orc.decode_step("gdn", orc.sketch_of(S0, Om), Om.T, toks, q)
    exact = orc.full_read_decode("gdn", S0, toks, q)
    assert np.abs(approx - exact).max() > 1e-3
    # and the difference is exactly S0^T (I - Om Om^T) q~
    x, _ = orc.effective_query("gdn", toks, q)
    np.testing.assert_allclose(exact - approx, S0.T @ (x - Om @ (Om.T @ x)), atol=1e-12)


# ---------------------------------------------------------------------------
# P3: replay of n tokens == n updates of one token
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("kind", KINDS)
def test_replay_equals_repeated_single_updates(kind):
    K, V, n, G = 10, 6, 7, 3
    rng = np.random.default_rng(8)
    toks = rand_tokens(rng, kind, n, K, V)
    S0 = rng.standard_normal((K, V))
    Om = rng.standard_normal((K, G))
    q = rng.standard_normal(K)
    S_all, U_all, o_all = orc.state_update(kind, S0, toks, Om, q)
    S = S0
    for tok in toks:
        S, U, _ = orc.state_update(kind, S, [tok], Om)
    np.testing.assert_allclose(S_all, S, rtol=0, atol=1e-13)
    np.testing.assert_allclose(U_all, U, rtol=0, atol=1e-13)
    np.testing.assert_allclose(U_all, S.T @ Om, rtol=0, atol=1e-13)
    np.testing.assert_allclose(o_all, S.T @ q, rtol=0, atol=1e-13)


# ---------------------------------------------------------------------------
# P4: empty buffer, and a no-op token
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("kind", KINDS)
def test_empty_buffer_output_is_U_C_q(kind):
    K, V, G = 6, 4, 2
    rng = np.random.default_rng(9)
    U = rng.standard_normal((V, G))
    C = rng.standard_normal((G, K))
    q = rng.standard_normal(K)
    np.testing.assert_allclose(orc.decode_step(kind, U, C, [], q), U @ (C @ q), atol=1e-14)
    noop = (rng.standard_normal(K), rng.standard_normal(V), np.float64(0.0),
            np.ones(K) if kind == "kda" else np.float64(1.0))
    np.testing.assert_allclose(orc.decode_step(kind, U, C, [noop], q), U @ (C @ q), atol=1e-14)


# ---------------------------------------------------------------------------
# P6: WY identities (Appendix C)
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("kind", ("gdn", "kda"))
def test_wy_form_equals_dense_product(kind):
    K, V, n = 5, 3, 4
    rng = np.random.default_rng(12)
    toks = rand_tokens(rng, kind, n, K, V)
    d_cum, pis, ls = orc.wy_factors(kind, toks)
    # base case printed in the paper: pi_1 = beta_1 (d_[1] * k_1)
    k1, _v, b1, dec1 = toks[0]
    d1 = dec1 if kind == "kda" else np.full(K, dec1)
    np.testing.assert_allclose(pis[0], b1 * d1 * k1, atol=1e-15)
    M = np.diag(d_cum[-1])
    for l_s, pi_s in zip(ls, pis):
        M = M - np.outer(l_s, pi_s)
    np.testing.assert_allclose(M, np.array(brute_prod(kind, toks, 1, n, K)), atol=1e-13)


@pytest.mark.parametrize("kind", KINDS)
def test_wy_effective_query_equals_sweep(kind):
    K, V, n = 12, 4, 6
    rng = np.random.default_rng(13)
    toks = rand_tokens(rng, kind, n, K, V, (3,))
    q = rng.standard_normal((3, K))
    x, _ = orc.effective_query(kind, toks, q)
    np.testing.assert_allclose(orc.wy_effective_query(kind, toks, q), x, atol=1e-13)
    if kind == "mamba2":       # q~ = d_[t] * q_t
        d = np.prod([t[3] for t in toks], axis=0)
        np.testing.assert_allclose(x, d[:, None] * q, atol=1e-14)


@pytest.mark.parametrize("kind", ("gdn", "kda"))
def test_projected_factors_give_C_qtilde_exactly(kind):
    K, V, n, G = 12, 4, 6, 3
    rng = np.random.default_rng(14)
    toks = rand_tokens(rng, kind, n, K, V)
    q = rng.standard_normal(K)
    C = rng.standard_normal((G, K))
    x, _ = orc.effective_query(kind, toks, q)
    np.testing.assert_allclose(orc.wy_coefficients(kind, toks, q, C), C @ x, atol=1e-13)


@pytest.mark.parametrize("kind", ("gdn", "kda"))
def test_projected_erase_vectors_are_C_times_the_erase_factors(kind):
    # f_s := C pi_s (the definition above Eq. 44), with pi_s from the recurrence of Eq. 42 that the dense transition
    # product pins; and the returned left factors / cumulative decay are those of the WY form
    K, V, n, G = 10, 3, 7, 4
    rng = np.random.default_rng(15)
    toks = rand_tokens(rng, kind, n, K, V, (2,))
    C = rng.standard_normal((2, G, K))
    d_cum, pis, ls = orc.wy_factors(kind, toks)
    fs, ls_f, d = orc.projected_erase_vectors(kind, toks, C)
    assert len(fs) == n
    for f_s, pi_s in zip(fs, pis):
        np.testing.assert_allclose(f_s, np.einsum("bgk,bk->bg", C, pi_s), atol=1e-13)
    for a, b in zip(ls_f, ls):
        np.testing.assert_allclose(a, b, atol=1e-15)
    np.testing.assert_allclose(d, d_cum[-1], atol=1e-15)
    # a prefix of the window gives the same vectors: f_s does not depend on later tokens
    fs5, _, _ = orc.projected_erase_vectors(kind, toks[:5], C)
    for a, b in zip(fs5, fs[:5]):
        np.testing.assert_allclose(a, b, atol=1e-15)


@pytest.mark.parametrize("kind", ("gdn", "kda"))
def test_stored_erase_vectors_with_rounding_stay_within_their_rounding_budget(kind):
    # With the vectors rounded to bfloat16 where they are stored, c_t moves by at most the sum over slots of the rounding
    # of each vector times |<l_s(t), q_t>|, plus what the rounded vectors pass on to later ones (second order); with the
    # identity as the store function nothing changes; and the decode step with such a store is U c_t + o^buffer.
    K, V, n, G = 12, 5, 7, 4
    rng = np.random.default_rng(19)
    toks = rand_tokens(rng, kind, n, K, V)
    q = rng.standard_normal(K)
    C = rng.standard_normal((G, K))
    U = rng.standard_normal((V, G))
    c0 = orc.wy_coefficients(kind, toks, q, C)
    np.testing.assert_allclose(orc.wy_coefficients(kind, toks, q, C, store=lambda f: f), c0, atol=0)
    cr = orc.wy_coefficients(kind, toks, q, C, store=orc.round_bf16)
    fs, ls, _ = orc.projected_erase_vectors(kind, toks, C)
    fr, _, _ = orc.projected_erase_vectors(kind, toks, C, store=orc.round_bf16)
    for f in fr:
        np.testing.assert_array_equal(f, orc.round_bf16(f))                    # stored values are bfloat16 values
    budget = sum(np.abs(fr_s - f_s) * abs(l_s @ q) for fr_s, f_s, l_s in zip(fr, fs, ls))
    assert np.all(np.abs(cr - c0) <= budget + 1e-12) and np.all(budget <= 2.0 ** -7 * sum(np.abs(f) * abs(l @ q) for f, l in zip(fs, ls)) + 1e-12)
    x, a = orc.effective_query(kind, toks, q)
    np.testing.assert_allclose(orc.decode_step(kind, U, C, toks, q, erase_store=orc.round_bf16),
                               U @ cr + orc.buffer_output(toks, a), atol=1e-13)
    np.testing.assert_allclose(orc.decode_step(kind, U, C, toks, q, erase_store=lambda f: f), orc.decode_step(kind, U, C, toks, q), atol=1e-12)


# ---------------------------------------------------------------------------
# Eq. 5-6: output error identity
# ---------------------------------------------------------------------------

def test_output_error_is_state_weighted_query_error():
    K, V, G = 9, 7, 3
    rng = np.random.default_rng(15)
    S0 = rng.standard_normal((K, V))
    Om = rng.standard_normal((K, G))
    x = rng.standard_normal(K)
    c = rng.standard_normal(G)
    lhs = np.sum((S0.T @ x - orc.sketch_of(S0, Om) @ c) ** 2)
    r = x - Om @ c
    np.testing.assert_allclose(lhs, r @ (S0 @ S0.T) @ r, rtol=1e-12)


# ---------------------------------------------------------------------------
# P7: offline fit (Appendix A.1, Eq. 8, Eq. 10)
# ---------------------------------------------------------------------------

def _spd(rng, K):
    A = rng.standard_normal((K, K))
    return A @ A.T / K + 0.1 * np.eye(K)


def test_fit_loss_equals_tail_eigenvalues_and_beats_random_bases():
    K, G, N = 10, 3, 500
    rng = np.random.default_rng(16)
    E0 = _spd(rng, K)
    Qt = rng.standard_normal((N, K)) @ rng.standard_normal((K, K))
    Om, lam = orc.fit_sketching_matrix(Qt, E0, G)
    assert np.all(np.diff(lam) <= 1e-12)
    # empirical loss of Eq. (8): mean over samples of the weighted least-squares residual,
    # solved sample by sample with a generic solver in the E0 metric
    w, Pm = np.linalg.eigh(E0)
    E_half = (Pm * np.sqrt(w)) @ Pm.T

    def loss(Omega):
        B = E_half @ Omega
        tot = 0.0
        for qi in Qt:
            z = E_half @ qi
            c, *_ = np.linalg.lstsq(B, z, rcond=None)
            tot += np.sum((z - B @ c) ** 2)
        return tot / N

    best = loss(Om)
    np.testing.assert_allclose(best, lam[G:].sum(), rtol=1e-9)
    for _ in range(5):
        assert loss(rng.standard_normal((K, G))) >= best - 1e-9


def test_offline_coefficient_map_collapses_to_PG_Ehalf():
    K, G, N = 8, 3, 300
    rng = np.random.default_rng(17)
    E0 = _spd(rng, K)
    Qt = rng.standard_normal((N, K))
    Om, _lam = orc.fit_sketching_matrix(Qt, E0, G)
    C = orc.offline_coefficient_map(Om, E0)
    w, Pm = np.linalg.eigh(E0)
    E_half = (Pm * np.sqrt(w)) @ Pm.T
    PG = E_half @ Om                                   # Omega* = E0^{-1/2} P_G
    np.testing.assert_allclose(PG.T @ PG, np.eye(G), atol=1e-10)
    np.testing.assert_allclose(C, PG.T @ E_half, atol=1e-9)
    np.testing.assert_allclose(C @ Om, np.eye(G), atol=1e-9)


def test_fit_with_identity_metric_is_textbook_pca():
    K, G, N = 12, 4, 400
    rng = np.random.default_rng(18)
    Qt = rng.standard_normal((N, 5)) @ rng.standard_normal((5, K)) + 0.01 * rng.standard_normal((N, K))
    Om, lam = orc.fit_sketching_matrix(Qt, np.eye(K), G)
    _u, s, vt = np.linalg.svd(Qt, full_matrices=False)
    np.testing.assert_allclose(lam[:G], (s[:G] ** 2) / N, rtol=1e-10)
    np.testing.assert_allclose(np.abs(Om.T @ vt[:G].T), np.eye(G), atol=1e-8)
    np.testing.assert_allclose(orc.offline_coefficient_map(Om, np.eye(K)), Om.T, atol=1e-10)
    # sign convention: largest-magnitude entry of every column is positive
    assert np.all(Om[np.abs(Om).argmax(axis=0), np.arange(G)] > 0)


def test_fit_with_singular_metric_uses_the_support():
    K, G, N = 6, 2, 200
    rng = np.random.default_rng(19)
    B = rng.standard_normal((K, 3))
    E0 = B @ B.T                                        # rank 3
    Qt = rng.standard_normal((N, K))
    Om, lam = orc.fit_sketching_matrix(Qt, E0, G)
    assert np.all(np.isfinite(Om))
    assert np.sum(lam > 1e-10) == 3
    # columns of Omega live in range(E0)
    null = np.linalg.svd(E0)[0][:, 3:]
    np.testing.assert_allclose(null.T @ Om, 0, atol=1e-9)


# ---------------------------------------------------------------------------
# P9: state-dependent coefficient map (Eq. 9, Appendix A.2.1)
# ---------------------------------------------------------------------------

def test_state_dependent_map_is_the_range_projection():
    K, V, G = 9, 7, 3
    rng = np.random.default_rng(20)
    S0 = rng.standard_normal((K, V))
    Om = rng.standard_normal((K, G))
    U = orc.sketch_of(S0, Om)
    C = orc.state_dependent_coefficient_map(S0, U)
    x = rng.standard_normal(K)
    o = S0.T @ x
    np.testing.assert_allclose(U.T @ (o - U @ (C @ x)), 0, atol=1e-11)
    Qu = np.linalg.qr(U)[0]
    np.testing.assert_allclose(U @ (C @ x), Qu @ (Qu.T @ o), atol=1e-11)


# ---------------------------------------------------------------------------
# P10: traffic model against the numbers printed in Tables 4-7
# ---------------------------------------------------------------------------

def _golden_rows():
    rows = []
    with open(os.path.join(GOLDEN, "traffic_reduction.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            t, m, K, V, e, W, G, val = line.split()
            rows.append((t, m, int(K), int(V), int(e), int(W), int(G), float(val)))
    return rows


def test_traffic_reduction_reproduces_printed_tables():
    rows = _golden_rows()
    assert len(rows) == 20
    for (_t, _m, K, V, e, W, G, val) in rows:
        assert abs(orc.traffic_reduction(K, V, G, W, bool(e)) - val) < 0.005 + 1e-9, (K, V, G, val)
    assert abs(orc.replay_traffic_reduction(16) - 32.0 / 17.0) < 1e-15
    assert round(orc.replay_traffic_reduction(16), 2) == 1.88
    # T_G = 2G(V + K + eW) and the G -> 0 limit is W (only the flush remains)
    assert orc.nonflush_read_bytes(128, 64, 5, 16, False) == 2 * 5 * 192
    assert orc.nonflush_read_bytes(128, 128, 7, 16, True) == 2 * 7 * 272
    assert abs(orc.traffic_reduction(128, 64, 0, 16, False) - 16.0) < 1e-12


# ---------------------------------------------------------------------------
# Algorithm 1 schedule
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("kind", KINDS)
def test_schedule_flush_outputs_are_exact_and_state_matches_recurrence(kind):
    K, V, G, L, T = 8, 6, 3, 4, 11
    rng = np.random.default_rng(21)
    toks = rand_tokens(rng, kind, T, K, V)
    qs = [rng.standard_normal(K) for _ in range(T)]
    S0 = rng.standard_normal((K, V))
    Om = np.linalg.qr(rng.standard_normal((K, G)))[0]
    outs, S_fin, U_fin, ring = orc.run_schedule(kind, S0, Om, Om.T, toks, qs, L)
    assert len(outs) == T and len(ring) == T % L
    S = S0
    for t in range(T):
        S = orc.transition(kind, S, *toks[t])
        if (t + 1) % L == 0:
            np.testing.assert_allclose(outs[t], S.T @ qs[t], atol=1e-12)      # flush step: exact
            S_at_flush = S
    np.testing.assert_allclose(S_fin, S_at_flush, atol=1e-12)
    np.testing.assert_allclose(U_fin, S_at_flush.T @ Om, atol=1e-12)
    # with the identity basis every step is exact
    outs_id, *_ = orc.run_schedule(kind, S0, np.eye(K), np.eye(K), toks, qs, L)
    S = S0
    for t in range(T):
        S = orc.transition(kind, S, *toks[t])
        np.testing.assert_allclose(outs_id[t], S.T @ qs[t], atol=1e-12)


# ---------------------------------------------------------------------------
# State-dependent coefficient maps (Appendix A.2.2, Eq. 26-37)
# ---------------------------------------------------------------------------

def _head(rng, K, V, G):
    S = rng.standard_normal((K, V)) * rng.uniform(0.2, 2.0, (K, 1))
    Om = np.linalg.qr(rng.standard_normal((K, G)))[0]
    return S, Om


def test_ridge_map_is_the_regularised_least_squares_solution():
    """c = C q~ minimises ||S^T (q~ - Omega c)||^2 / mu + lam ||c||^2 (Eq. 28-29 carried back to the original
    coordinates, which the orthogonal change of basis preserves): a library least-squares solve of the stacked
    system [S^T Omega / sqrt(mu); sqrt(lam) I] c = [S^T q~ / sqrt(mu); 0] gives the same vector."""
    rng = np.random.default_rng(11)
    for (K, V, G, lam) in [(16, 12, 5, 0.1), (24, 8, 8, 0.1), (10, 10, 3, 2.5)]:
        S, Om = _head(rng, K, V, G)
        C = orc.ridge_coefficient_map(S, Om, lam)
        mu = float((S * S).sum()) / K
        for _ in range(3):
            q = rng.standard_normal(K)
            A = np.concatenate([S.T @ Om / np.sqrt(mu), np.sqrt(lam) * np.eye(G)])
            b = np.concatenate([S.T @ q / np.sqrt(mu), np.zeros(G)])
            c_ls = np.linalg.lstsq(A, b, rcond=None)[0]
            np.testing.assert_allclose(C @ q, c_ls, atol=1e-10)


def test_ridge_map_tends_to_the_range_projection_without_ridge():
    """lam -> 0 with a full-column-rank sketch: the map of Eq. 9, and U c is the orthogonal projection of the
    exact read onto range(U) (Eq. 25)."""
    rng = np.random.default_rng(12)
    S, Om = _head(rng, 20, 14, 6)
    U = S.T @ Om
    C0 = orc.ridge_coefficient_map(S, Om, 1e-13)
    np.testing.assert_allclose(C0, orc.state_dependent_coefficient_map(S, U), atol=1e-7)
    q = rng.standard_normal(20)
    resid = S.T @ q - U @ (C0 @ q)
    np.testing.assert_allclose(U.T @ resid, 0.0, atol=1e-7)


def test_state_dependent_maps_do_not_depend_on_the_orthogonal_completion():
    """R completes Omega to an orthogonal matrix; any completion must give the same map.  A second completion is
    obtained by rotating the complement, and the maps are rebuilt from scratch in those coordinates."""
    rng = np.random.default_rng(13)
    K, V, G = 14, 9, 5
    S, Om = _head(rng, K, V, G)
    R1 = orc._orthogonal_completion(Om)
    W = np.linalg.qr(rng.standard_normal((K - G, K - G)))[0]
    R2 = np.concatenate([R1[:G], W @ R1[G:]])
    np.testing.assert_allclose(R2 @ R2.T, np.eye(K), atol=1e-12)
    lam = 0.1
    mu = float((S * S).sum()) / K
    J = np.eye(K)[:, :G]
    for name, C in (("ridge", orc.ridge_coefficient_map(S, Om, lam)), ("pivot", orc.pivot_coefficient_map(S, Om, lam, 3))):
        Sp = R2 @ S
        H = Sp @ Sp.T / mu
        if name == "ridge":
            C2 = np.linalg.solve(J.T @ H @ J + lam * np.eye(G), J.T @ H) @ R2
        else:
            Uq = np.linalg.qr((Sp.T @ J)[:, :3])[0]
            L = Sp @ Uq / np.sqrt(mu)
            d = np.maximum(np.diag(H) - (L * L).sum(1), 0.0)
            Hh = L @ L.T + np.diag(d)
            C2 = np.linalg.solve(J.T @ Hh @ J + lam * np.eye(G), J.T @ Hh) @ R2
        np.testing.assert_allclose(C, C2, atol=1e-10, err_msg=name)


def test_pivot_map_woodbury_step_equals_a_dense_solve_and_keeps_the_diagonal():
    """(D_G + L_G L_G^T)^{-1} through the p x p Woodbury system equals a dense G x G solve with H^ = L L^T + Diag(d)
    (Eq. 34-37), and H^ keeps the diagonal of H (Eq. 33)."""
    rng = np.random.default_rng(14)
    for (K, V, G, P) in [(16, 12, 7, 4), (12, 20, 5, 2), (18, 6, 6, 4)]:
        S, Om = _head(rng, K, V, G)
        lam = 0.1
        R, mu, Q, L, d = orc.pivot_metric_factors(S, Om, P)
        Sp = R @ S
        H = Sp @ Sp.T / mu
        np.testing.assert_allclose(Q.T @ Q, np.eye(min(G, P)), atol=1e-12)
        # Q spans the first p sketch columns
        Up = (S.T @ Om)[:, :min(G, P)]
        np.testing.assert_allclose(Q @ (Q.T @ Up), Up, atol=1e-10)
        Hh = L @ L.T + np.diag(d)
        np.testing.assert_allclose(np.diag(Hh), np.diag(H), atol=1e-12)
        J = np.eye(K)[:, :G]
        dense = np.linalg.solve(J.T @ Hh @ J + lam * np.eye(G), J.T @ Hh) @ R
        np.testing.assert_allclose(orc.pivot_coefficient_map(S, Om, lam, P), dense, atol=1e-10)


def test_pivot_map_with_all_sketch_columns_as_pivots_is_the_ridge_map():
    """P >= G: Q spans range(U), so L L^T reproduces every block of H the solve uses and the residual diagonal on the
    retained coordinates vanishes: the approximation is exact."""
    rng = np.random.default_rng(15)
    S, Om = _head(rng, 16, 11, 4)
    for P in (4, 6):
        np.testing.assert_allclose(orc.pivot_coefficient_map(S, Om, 0.1, P), orc.ridge_coefficient_map(S, Om, 0.1), atol=1e-10)
    assert np.abs(orc.pivot_coefficient_map(S, Om, 0.1, 2) - orc.ridge_coefficient_map(S, Om, 0.1)).max() > 1e-3


def test_pivot_map_handles_dependent_pivot_columns_and_the_zero_state():
    rng = np.random.default_rng(16)
    K, V, G = 10, 8, 4
    S, Om = _head(rng, K, V, G)
    # make the second sketch column a multiple of the first: S^T (omega_2 - 3 omega_1) = 0
    w = Om[:, 1] - 3.0 * Om[:, 0]
    S = S - np.outer(w, w @ S) / (w @ w)
    R, mu, Q, L, d = orc.pivot_metric_factors(S, Om, 4)
    assert np.allclose(Q[:, 1], 0.0) and np.linalg.matrix_rank(Q) == 3
    assert np.all(np.isfinite(orc.pivot_coefficient_map(S, Om)))
    Z = np.zeros((K, V))
    assert np.allclose(orc.pivot_coefficient_map(Z, Om), 0.0) and np.allclose(orc.ridge_coefficient_map(Z, Om), 0.0)


def test_sketch_form_maps_equal_the_appendix_forms_at_the_exact_sketch():
    """The restatements in terms of (S_0, U, Omega) that define the map built from a stored sketch: at U = S_0^T Omega
    they are the appendix's maps (which are pinned above); with a dependent pivot column and the zero state too; and
    the ridge form at a perturbed U is still the regularised least-squares solution for that U."""
    rng = np.random.default_rng(18)
    for (K, V, G, P, lam) in [(16, 12, 5, 4, 0.1), (24, 8, 8, 4, 0.1), (12, 10, 3, 4, 0.7), (20, 16, 6, 2, 0.1)]:
        S, Om = _head(rng, K, V, G)
        U = S.T @ Om
        np.testing.assert_allclose(orc.ridge_coefficient_map_from_sketch(S, U, lam), orc.ridge_coefficient_map(S, Om, lam),
                                   rtol=0, atol=1e-10)
        np.testing.assert_allclose(orc.pivot_coefficient_map_from_sketch(S, U, Om, lam, P),
                                   orc.pivot_coefficient_map(S, Om, lam, P), rtol=0, atol=1e-10)
        Cb = orc.coefficient_maps(S[None], Om[None], "pivot", lam, P, U=U[None])
        np.testing.assert_allclose(Cb[0], orc.pivot_coefficient_map(S, Om, lam, P), atol=1e-10)
        # a sketch that is not exactly S^T Omega (as after rounding): the ridge form solves the least-squares problem of that U
        Up = U * (1.0 + 2.0 ** -8 * (rng.random(U.shape) < 0.3))
        C = orc.ridge_coefficient_map_from_sketch(S, Up, lam)
        mu = float((S * S).sum()) / K
        q = rng.standard_normal(K)
        A = np.concatenate([Up / np.sqrt(mu), np.sqrt(lam) * np.eye(G)])
        b = np.concatenate([S.T @ q / np.sqrt(mu), np.zeros(G)])
        np.testing.assert_allclose(C @ q, np.linalg.lstsq(A, b, rcond=None)[0], atol=1e-10)
    K, V, G = 10, 8, 4
    S, Om = _head(rng, K, V, G)
    w = Om[:, 1] - 3.0 * Om[:, 0]
    S = S - np.outer(w, w @ S) / (w @ w)
    np.testing.assert_allclose(orc.pivot_coefficient_map_from_sketch(S, S.T @ Om, Om), orc.pivot_coefficient_map(S, Om), atol=1e-9)
    Z = np.zeros((K, V))
    assert np.allclose(orc.pivot_coefficient_map_from_sketch(Z, Z.T @ Om, Om), 0.0)
    assert np.allclose(orc.ridge_coefficient_map_from_sketch(Z, Z.T @ Om), 0.0)


def test_pivot_map_brute_force_on_tiny_heads():
    """K, V <= 4 with Python loops only: rotate the state, build mu, H, the Gram-Schmidt basis of the first p sketch
    columns, L, d and H^ entry by entry, and solve the G x G normal equations by hand-written elimination."""
    rng = np.random.default_rng(17)
    K, V, G, P, lam = 4, 3, 3, 2, 0.1
    S, Om = _head(rng, K, V, G)
    R = orc._orthogonal_completion(Om)
    Sp = [[sum(R[i][l] * S[l][j] for l in range(K)) for j in range(V)] for i in range(K)]
    mu = sum(Sp[i][j] ** 2 for i in range(K) for j in range(V)) / K
    Hd = [sum(Sp[i][j] ** 2 for j in range(V)) / mu for i in range(K)]
    # Gram-Schmidt on the first two sketch columns (column g of the sketch is row g of S')
    u1 = Sp[0][:]
    n1 = sum(x * x for x in u1) ** 0.5
    q1 = [x / n1 for x in u1]
    r12 = sum(a * b for a, b in zip(q1, Sp[1]))
    u2 = [b - r12 * a for a, b in zip(q1, Sp[1])]
    n2 = sum(x * x for x in u2) ** 0.5
    q2 = [x / n2 for x in u2]
    Lm = [[sum(Sp[i][j] * q[j] for j in range(V)) / mu ** 0.5 for q in (q1, q2)] for i in range(K)]
    dd = [max(Hd[i] - Lm[i][0] ** 2 - Lm[i][1] ** 2, 0.0) for i in range(K)]
    Hh = [[Lm[i][0] * Lm[j][0] + Lm[i][1] * Lm[j][1] + (dd[i] if i == j else 0.0) for j in range(K)] for i in range(K)]
    q = list(rng.standard_normal(K))
    x = [sum(R[i][l] * q[l] for l in range(K)) for i in range(K)]
    A = [[Hh[i][j] + (lam if i == j else 0.0) for j in range(G)] for i in range(G)]
    b = [sum(Hh[i][j] * x[j] for j in range(K)) for i in range(G)]
    for col in range(G):                                   # Gaussian elimination, no pivoting needed (SPD)
        for row in range(col + 1, G):
            f = A[row][col] / A[col][col]
            for j in range(col, G):
                A[row][j] -= f * A[col][j]
            b[row] -= f * b[col]
    c = [0.0] * G
    for i in range(G - 1, -1, -1):
        c[i] = (b[i] - sum(A[i][j] * c[j] for j in range(i + 1, G))) / A[i][i]
    np.testing.assert_allclose(orc.pivot_coefficient_map(S, Om, lam, P) @ np.array(q), c, atol=1e-10)


@pytest.mark.parametrize("kind", KINDS)
def test_schedule_with_state_dependent_map_rebuilds_it_at_every_flush(kind):
    """run_schedule_state_dependent: the map in force during a window is the one of the state at the window's start;
    flush outputs are exact; with all sketch columns as pivots and no ridge the sketch read is the projection of the
    exact read onto range(U)."""
    rng = np.random.default_rng(18)
    N, K, V, G, L = 3, 8, 6, 3, 4
    S0 = rng.standard_normal((N, K, V))
    Om = np.stack([np.linalg.qr(rng.standard_normal((K, G)))[0] for _ in range(N)])
    toks = rand_tokens(rng, kind, 2 * L + 1, K, V, lead=(N,))
    qs = [rng.standard_normal((N, K)) for _ in toks]
    outs, S, U, C = orc.run_schedule_state_dependent(kind, S0, Om, toks, qs, L, "pivot", lam=0.1, P=2)
    # replay by hand
    St = S0.copy()
    Sw = S0.copy()
    for t, (tok, q) in enumerate(zip(toks, qs)):
        St = orc.transition(kind, St, *tok)
        exact = orc.exact_read(St, q)
        if t % L == L - 1:
            np.testing.assert_allclose(outs[t], exact, atol=1e-10)
            Sw = St.copy()
        else:
            ring = toks[(t // L) * L: t + 1]
            Cw = np.stack([orc.pivot_coefficient_map(Sw[i], Om[i], 0.1, 2) for i in range(N)])
            want = orc.decode_step(kind, orc.sketch_of(Sw, Om), Cw, ring, q)
            np.testing.assert_allclose(outs[t], want, atol=1e-10)
    np.testing.assert_allclose(C, np.stack([orc.pivot_coefficient_map(Sw[i], Om[i], 0.1, 2) for i in range(N)]), atol=1e-12)


def test_round_bf16_is_round_to_nearest_even_on_the_top_16_bits():
    """Pinned against hand-picked values: bfloat16 keeps 8 significand bits (spacing 2^-7 in [1, 2))."""
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 2.0 ** -7, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, -0.3, 0.0, 3.0e38])
    want = np.array([1.0, 1.0, 1.0 + 2.0 ** -7, 1.0 + 2.0 ** -6, 1.0 + 2.0 ** -7, -0.30078125, 0.0, 226.0 / 128.0 * 2.0 ** 127])
    got = orc.round_bf16(x)
    np.testing.assert_allclose(got, want, rtol=1e-7)
    # idempotent, and within half a spacing of the input
    np.testing.assert_array_equal(orc.round_bf16(got), got)
    rng = np.random.default_rng(21)
    y = rng.standard_normal(1000)
    assert np.all(np.abs(orc.round_bf16(y) - y) <= np.abs(y) * 2.0 ** -8)
