"""Pins for the CPU oracle: facts fixed by the paper or by mathematics.

Each pin is a function ``pin(orc)`` that raises AssertionError when the oracle
build ``orc`` (an ``oracle.OracleLib``) violates it.  None of them re-types the
oracle's recurrence: they use brute-force inverses, closed forms, textbook
reductions, invariants and a second evaluation order.  ``test_oracle_pins.py``
runs them on the committed oracle; ``test_oracle_mutants.py`` checks that each
planted mistake in a copy of the oracle trips at least one of them.
"""
import numpy as np

IDENT = 1  # oracle.IDENTITY_MAP
EPS = 1e-4


def _phi(x):
    """ELU(x)+1 (Section 3.3)."""
    return np.where(x > 0, x + 1.0, np.exp(np.minimum(x, 0.0)))


def _khat(k, flags):
    kf = k if flags & IDENT else _phi(k)
    return kf / np.linalg.norm(kf, axis=-1, keepdims=True)


def _unit(x):
    return x / np.linalg.norm(x, axis=-1, keepdims=True)


def _rand(seed, T, dk, dv):
    g = np.random.default_rng(seed)
    return g.standard_normal((T, dk)), g.standard_normal((T, dk)), g.standard_normal((T, dv)), g


def _u_variants(g, T, dk):
    ru = _unit(g.standard_normal((T, dk)))
    return {"khat": None, "unit": ru, "unit_over_sqrt_d": ru / np.sqrt(dk),
            "free": 0.7 * g.standard_normal((T, dk))}


# --------------------------------------------------------------------------
# A-chain: A_t is exactly the inverse of M_t = lambda*I + sum u u^T
# (Section 1.2; Eq. "penalty"; Eq. "A-covariance")
# --------------------------------------------------------------------------
def pin_A_is_brute_force_inverse(orc):
    for dk, T, lam, flags, seed in [(2, 5, 0.1, 0, 1), (3, 17, 1.0, IDENT, 2), (5, 64, 0.1, IDENT, 3),
                                    (8, 33, 1.0, 0, 4), (16, 64, 0.1, 0, 5), (16, 40, 2.5, IDENT, 6)]:
        q, k, v, g = _rand(seed, T, dk, dk)
        for name, u in _u_variants(g, T, dk).items():
            r = orc.forward_trace(q, k, v, lam, u=u, flags=flags)
            used = _khat(k, flags) if u is None else u
            M = lam * np.eye(dk)
            for t in range(T):
                M = M + np.outer(used[t], used[t])
                ref = np.linalg.inv(M)
                err = np.abs(r.trace["A"][t] - ref).max() / np.abs(ref).max()
                assert err < 1e-10, (dk, T, lam, name, t, err)
            assert np.allclose(r.A_T, r.trace["A"][-1], rtol=0, atol=0)


def pin_A_invariants(orc):
    """delta in [1, 1+1/lambda]; A symmetric, eigenvalues in [1/(lambda+t), 1/lambda];
    tr(A_t^{-1}) = d*lambda + t; A_t <= A_{t-1} (Loewner).  Unit-norm u (Eq. "penalty")."""
    for dk, T, lam, flags, seed in [(4, 30, 0.1, 0, 11), (12, 50, 1.0, IDENT, 12)]:
        q, k, v, g = _rand(seed, T, dk, dk)
        for u in (None, _unit(g.standard_normal((T, dk)))):
            r = orc.forward_trace(q, k, v, lam, u=u, flags=flags)
            d = r.trace["delta"]
            assert np.all(d >= 1.0 - 1e-12) and np.all(d <= 1.0 + 1.0 / lam + 1e-12)
            prev = np.eye(dk) / lam
            for t in range(T):
                A = r.trace["A"][t]
                assert np.abs(A - A.T).max() < 1e-13 * np.abs(A).max() + 1e-15
                w = np.linalg.eigvalsh(0.5 * (A + A.T))
                assert w.min() >= 1.0 / (lam + t + 1) - 1e-12
                assert w.max() <= 1.0 / lam + 1e-12
                assert abs(np.trace(np.linalg.inv(A)) - (dk * lam + t + 1)) < 1e-8 * (dk * lam + t + 1)
                assert np.linalg.eigvalsh(prev - A).min() > -1e-12
                prev = A


def pin_delta_value(orc):
    """delta_t = 1 + u^T A_{t-1} u with the brute-force A_{t-1} (Eq. "sm")."""
    dk, T, lam = 6, 12, 0.5
    q, k, v, g = _rand(21, T, dk, dk)
    u = 0.9 * g.standard_normal((T, dk))
    r = orc.forward_trace(q, k, v, lam, u=u, flags=IDENT)
    M = lam * np.eye(dk)
    for t in range(T):
        ref = 1.0 + u[t] @ np.linalg.inv(M) @ u[t]
        assert abs(r.trace["delta"][t] - ref) < 1e-10 * ref
        M += np.outer(u[t], u[t])


# --------------------------------------------------------------------------
# write direction (Eq. "s-update"; Appendix A.1 "post-update A_t")
# --------------------------------------------------------------------------
def pin_alpha_from_post_update_A(orc):
    for flags in (0, IDENT):
        dk, T, lam = 7, 20, 0.3
        q, k, v, g = _rand(31 + flags, T, dk, dk)
        u = _unit(g.standard_normal((T, dk)))       # u != k_hat: pre- and post-update differ
        r = orc.forward_trace(q, k, v, lam, u=u, flags=flags)
        kh = _khat(k, flags)
        assert np.abs(r.trace["khat"] - kh).max() < 1e-14
        M = lam * np.eye(dk)
        for t in range(T):
            M += np.outer(u[t], u[t])
            a = np.linalg.solve(M, kh[t])
            a /= np.linalg.norm(a)
            assert np.abs(r.trace["alpha"][t] - a).max() < 1e-11, t
            c = a @ kh[t]
            assert 0.0 < c <= 1.0 + 1e-14
        assert np.abs(np.linalg.norm(r.trace["alpha"], axis=1) - 1).max() < 1e-14
        assert np.abs(np.linalg.norm(r.trace["khat"], axis=1) - 1).max() < 1e-14


# --------------------------------------------------------------------------
# S-chain closed forms
# --------------------------------------------------------------------------
def pin_first_step_closed_form(orc):
    """From S_0=0, A_0=I/lambda, u=k_hat: A_1 = I/lambda - kk^T/(lambda(lambda+1)),
    alpha_1 = k_hat, S_1 = v k_hat^T; o_1 = v (k_hat.q) [identity], v/||phi(k)|| [paper]."""
    dk, dv, lam = 5, 3, 0.1
    q, k, v, _ = _rand(41, 1, dk, dv)
    for flags in (0, IDENT):
        r = orc.forward_trace(q, k, v, lam, flags=flags)
        kh = _khat(k, flags)[0]
        A1 = np.eye(dk) / lam - np.outer(kh, kh) / (lam * (lam + 1))
        assert np.abs(r.A_T - A1).max() < 1e-13
        assert np.abs(r.trace["alpha"][0] - kh).max() < 1e-14
        assert np.abs(r.S_T - np.outer(v[0], kh)).max() < 1e-14
        if flags & IDENT:
            assert np.abs(r.out[0] - v[0] * (kh @ q[0])).max() < 1e-14
        else:
            assert np.abs(r.out[0] - v[0] / np.linalg.norm(_phi(k[0]))).max() < 1e-14
            assert np.abs(r.z_T - _phi(k[0])).max() < 1e-15


def pin_orthonormal_keys_exact_recall(orc):
    """Orthonormal keys (any positive scale), identity map, u=k_hat, T=d: A_T =
    Q diag(1/(lambda+1)) Q^T, alpha=k_hat, S_T k_hat_i = v_i (Proposition 3's special case)."""
    dk, dv, lam = 8, 5, 0.1
    g = np.random.default_rng(51)
    Q, _ = np.linalg.qr(g.standard_normal((dk, dk)))
    scale = g.uniform(0.5, 3.0, size=dk)
    k = (Q * scale).T.copy()                # row t = scale_t * Q[:, t]
    v = g.standard_normal((dk, dv))
    q = k[::-1].copy()                      # query the stored keys in reverse order
    r = orc.forward_trace(q, k, v, lam, flags=IDENT)
    assert np.abs(r.S_T @ Q - v.T).max() < 1e-13
    assert np.abs(r.A_T - np.eye(dk) / (lam + 1)).max() < 1e-13
    # columns are written once and never touched again: S_t = sum_{s<=t} v_s q_s^T
    for t in range(dk):
        assert np.abs(r.trace["S"][t] - v[:t + 1].T @ Q[:, :t + 1].T).max() < 1e-13
    # a later query for an already stored key returns its value times the key scale
    for t in range(dk):
        j = dk - 1 - t
        expect = (v[j] * scale[j]) if j <= t else 0.0 * v[j]
        assert np.abs(r.out[t] - expect).max() < 1e-12


def pin_repeated_key(orc):
    """Same key every step, u=k_hat: A_t = I/lambda - kk^T t/(lambda(lambda+t)), S_t = v_t k_hat^T."""
    dk, dv, T, lam = 6, 4, 15, 0.7
    g = np.random.default_rng(61)
    k = np.tile(g.standard_normal((1, dk)), (T, 1))
    v = g.standard_normal((T, dv))
    q = g.standard_normal((T, dk))
    for flags in (0, IDENT):
        r = orc.forward_trace(q, k, v, lam, flags=flags)
        kh = _khat(k[:1], flags)[0]
        for t in range(T):
            n = t + 1
            At = np.eye(dk) / lam - np.outer(kh, kh) * n / (lam * (lam + n))
            assert np.abs(r.trace["A"][t] - At).max() < 1e-12
            assert np.abs(r.trace["S"][t] - np.outer(v[t], kh)).max() < 1e-12


def pin_zero_u_is_normalised_delta_rule(orc):
    """u = 0 keeps A = A_0; with A_0 = I/lambda, alpha = k_hat and S follows the
    normalised LMS / delta rule S += (v - S k_hat) k_hat^T (Remark, Section 4.4)."""
    dk, dv, T, lam = 9, 7, 40, 0.1
    q, k, v, g = _rand(71, T, dk, dv)
    r = orc.forward_trace(q, k, v, lam, u=np.zeros((T, dk)), flags=IDENT)
    assert np.abs(r.A_T - np.eye(dk) / lam).max() == 0.0
    S = np.zeros((dv, dk))
    for t in range(T):
        kh = k[t] / np.linalg.norm(k[t])
        S = S + np.outer(v[t] - S @ kh, kh)
        assert np.abs(r.trace["S"][t] - S).max() < 1e-12
        assert np.abs(r.out[t] - S @ q[t]).max() < 1e-12
    # fixed anisotropic A_0: alpha is A_0 k_hat normalised
    B0 = g.standard_normal((dk, dk))
    A0 = B0 @ B0.T + 0.5 * np.eye(dk)
    r = orc.forward_trace(q, k, v, lam, u=np.zeros((T, dk)), A0=A0, flags=IDENT)
    kh = _khat(k, IDENT)
    al = _unit(kh @ A0)          # A0 symmetric
    assert np.abs(r.trace["alpha"] - al).max() < 1e-13


def pin_associative_composition(orc):
    """Second evaluation order (Section 3.4, with the map acting on the right):
    S_t = S_{t-1} R_t + G_t, R_t = I - k_hat alpha^T, G_t = v alpha^T; pairs compose
    as (R_l, G_l) then (R_r, G_r) -> (R_l R_r, G_l R_r + G_r).  A balanced tree over
    the steps must reproduce the sequential S_T."""
    dk, dv, T, lam = 6, 4, 37, 0.2
    q, k, v, g = _rand(81, T, dk, dv)
    u = _unit(g.standard_normal((T, dk)))
    S0 = g.standard_normal((dv, dk))
    r = orc.forward_trace(q, k, v, lam, u=u, S0=S0, flags=0)
    kh, al = _khat(k, 0), r.trace["alpha"]
    items = [(np.eye(dk) - np.outer(kh[t], al[t]), np.outer(v[t], al[t])) for t in range(T)]
    while len(items) > 1:
        nxt = []
        for i in range(0, len(items) - 1, 2):
            (Rl, Gl), (Rr, Gr) = items[i], items[i + 1]
            nxt.append((Rl @ Rr, Gl @ Rr + Gr))
        if len(items) % 2:
            nxt.append(items[-1])
        items = nxt
    R, G = items[0]
    assert np.abs(S0 @ R + G - r.S_T).max() < 1e-11


def pin_proposition_1(orc):
    """||S_t - S_{t-1}||_F = ||e_t||, ||S_t||_F <= ||S_0||_F + sum ||e_s||, and
    the residual identity v_t - S_t k_hat_t = (1 - alpha.k_hat) e_t."""
    dk, dv, T, lam = 10, 6, 60, 0.1
    q, k, v, g = _rand(91, T, dk, dv)
    S0 = 0.3 * g.standard_normal((dv, dk))
    for flags in (0, IDENT):
        r = orc.forward_trace(q, k, v, lam, S0=S0, flags=flags)
        prev, acc = S0, np.linalg.norm(S0)
        for t in range(T):
            St, e = r.trace["S"][t], r.trace["e"][t]
            assert abs(np.linalg.norm(St - prev) - np.linalg.norm(e)) < 1e-12
            acc += np.linalg.norm(e)
            assert np.linalg.norm(St) <= acc + 1e-12
            kh = r.trace["khat"][t]
            assert np.abs(e - (v[t] - prev @ kh)).max() < 1e-12           # residual uses S_{t-1}
            c = r.trace["alpha"][t] @ kh
            assert np.abs((v[t] - St @ kh) - (1 - c) * e).max() < 1e-11
            assert np.abs(St - prev - np.outer(e, r.trace["alpha"][t])).max() < 1e-13
            prev = St


def pin_readout(orc):
    """identity: o_t = S_t q_t;  paper: o_t = S_t phi(q_t) / max(phi(q_t).sum_{s<=t} phi(k_s), eps)."""
    dk, dv, T, lam = 7, 5, 25, 0.1
    q, k, v, g = _rand(101, T, dk, dv)
    u = _unit(g.standard_normal((T, dk)))
    r = orc.forward_trace(q, k, v, lam, u=u, flags=IDENT)
    for t in range(T):
        assert np.abs(r.out[t] - r.trace["S"][t] @ q[t]).max() < 1e-12
    assert np.all(r.trace["den"] == 1.0)
    z0 = np.abs(g.standard_normal(dk))
    r = orc.forward_trace(q, k, v, lam, u=u, z0=z0, flags=0)
    fk, fq = _phi(k), _phi(q)
    for t in range(T):
        den = max(fq[t] @ (z0 + fk[:t + 1].sum(0)), EPS)
        assert abs(r.trace["den"][t] - den) < 1e-12 * den
        assert np.abs(r.out[t] - r.trace["S"][t] @ fq[t] / den).max() < 1e-12
    assert np.abs(r.z_T - (z0 + fk.sum(0))).max() < 1e-12


def pin_feature_map_values(orc):
    """phi(x) = x+1 for x>0, exp(x) for x<=0, read back through z_T after one token."""
    xs = np.array([[-30.0, -2.0, -1e-9, 0.0, 1e-9, 0.5, 3.0, 40.0]])
    r = orc.forward_trace(xs, xs, np.zeros((1, 2)), 1.0, flags=0)
    expect = np.array([np.exp(-30.0), np.exp(-2.0), np.exp(-1e-9), 1.0, 1.0 + 1e-9, 1.5, 4.0, 41.0])
    assert np.abs(r.z_T - expect).max() < 1e-15 * 41


def pin_eps_guards(orc):
    """A zero key (identity map) gives k_hat = 0, alpha = 0, no update and no NaN; a
    tiny readout denominator is clamped to eps (Section 5.3)."""
    dk, dv, lam = 4, 3, 1.0
    g = np.random.default_rng(111)
    k = g.standard_normal((3, dk)); k[1] = 0.0
    v = g.standard_normal((3, dv)); q = g.standard_normal((3, dk))
    r = orc.forward_trace(q, k, v, lam, flags=IDENT)
    assert np.all(np.isfinite(r.out)) and np.all(np.isfinite(r.A_T))
    assert np.all(r.trace["khat"][1] == 0) and np.all(r.trace["alpha"][1] == 0)
    assert np.all(r.trace["S"][1] == r.trace["S"][0]) and np.all(r.trace["A"][1] == r.trace["A"][0])
    # paper mode: phi(-60) ~ 1e-26 on every coordinate -> denominator below eps
    kk = np.full((1, dk), -60.0)
    r = orc.forward_trace(kk, kk, np.ones((1, dv)), lam, flags=0)
    assert r.trace["den"][0] == EPS
    assert np.all(np.isfinite(r.out))


def pin_state_carry(orc):
    """forward(T) equals forward(T1) then forward(T-T1) with (S, A, z) carried."""
    B, H, T, dk, dv, lam = 2, 3, 23, 6, 4, 0.1
    g = np.random.default_rng(121)
    q = g.standard_normal((B, H, T, dk)); k = g.standard_normal((B, H, T, dk))
    v = g.standard_normal((B, H, T, dv)); u = _unit(g.standard_normal((B, H, T, dk)))
    for flags in (0, IDENT):
        for uu in (None, u):
            full = orc.forward(q, k, v, lam, u=uu, in_dtype=2, flags=flags)
            for T1 in (0, 1, 9, T):
                a = orc.forward(q[:, :, :T1], k[:, :, :T1], v[:, :, :T1], lam,
                                u=None if uu is None else uu[:, :, :T1], in_dtype=2, flags=flags)
                b = orc.forward(q[:, :, T1:], k[:, :, T1:], v[:, :, T1:], lam,
                                u=None if uu is None else uu[:, :, T1:], in_dtype=2, flags=flags,
                                S0=a.S_T, A0=a.A_T, z0=a.z_T)
                cat = np.concatenate([a.out, b.out], axis=2)
                assert np.abs(cat - full.out).max() < 1e-12
                assert np.abs(b.S_T - full.S_T).max() < 1e-12
                assert np.abs(b.A_T - full.A_T).max() < 1e-12
                assert np.abs(b.z_T - full.z_T).max() < 1e-12


def pin_units_layout_threads_dtypes(orc):
    """The batched entry point treats every (b,h) as an independent unit in [B,H,T,d]
    order, threads do not change results, and f32 / bf16 storage is widened exactly."""
    B, H, T, dk, dv, lam = 2, 2, 11, 4, 3, 1.0
    g = np.random.default_rng(131)
    q = g.standard_normal((B, H, T, dk)).astype(np.float32)
    k = g.standard_normal((B, H, T, dk)).astype(np.float32)
    v = g.standard_normal((B, H, T, dv)).astype(np.float32)
    r1 = orc.forward(q, k, v, lam, in_dtype=0, n_threads=1)
    r3 = orc.forward(q, k, v, lam, in_dtype=0, n_threads=3)
    r64 = orc.forward(q.astype(np.float64), k.astype(np.float64), v.astype(np.float64), lam, in_dtype=2)
    for a, b in ((r1, r3), (r1, r64)):
        assert np.array_equal(a.out, b.out) and np.array_equal(a.S_T, b.S_T)
        assert np.array_equal(a.A_T, b.A_T) and np.array_equal(a.z_T, b.z_T)
    for b in range(B):
        for h in range(H):
            one = orc.forward_trace(q[b, h], k[b, h], v[b, h], lam, in_dtype=0)
            assert np.array_equal(one.out, r1.out[b, h]) and np.array_equal(one.S_T, r1.S_T[b, h])
    # bf16: keep the upper 16 bits of the f32 pattern; the oracle must see exactly that value
    def to_bf16_bits(x):
        return (x.view(np.uint32) >> 16).astype(np.uint16)
    def from_bits(b):
        return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    qb, kb, vb = to_bf16_bits(q), to_bf16_bits(k), to_bf16_bits(v)
    rb = orc.forward(qb, kb, vb, lam, in_dtype=1)
    rr = orc.forward(from_bits(qb), from_bits(kb), from_bits(vb), lam, in_dtype=2)
    assert np.array_equal(rb.out, rr.out) and np.array_equal(rb.A_T, rr.A_T)


def pin_jacobian_spectrum(orc):
    """J_t = I - alpha k_hat^T (Proposition 2): eigenvalues are 1 (d-1 times) and 1-c with
    c = alpha.k_hat in (0,1], so the spectral radius is exactly 1.  Its largest singular
    value is sqrt((3-2c+sqrt(5-4c))/2), which is 1 only when c = 1 and is below the golden
    ratio otherwise; the paper's claim of 1 for every t holds for the radius, not the norm."""
    dk, T, lam = 8, 30, 0.1
    q, k, v, g = _rand(141, T, dk, dk)
    r = orc.forward_trace(q, k, v, lam, u=_unit(g.standard_normal((T, dk))), flags=0)
    for t in range(T):
        al, kh = r.trace["alpha"][t], r.trace["khat"][t]
        c = al @ kh
        assert 0 < c <= 1 + 1e-14
        J = np.eye(dk) - np.outer(al, kh)
        ev = np.sort(np.linalg.eigvals(J).real)
        assert abs(ev[0] - (1 - c)) < 1e-9 and np.abs(ev[1:] - 1).max() < 1e-7
        smax = np.linalg.norm(J, 2)
        assert abs(smax - np.sqrt((3 - 2 * c + np.sqrt(5 - 4 * c)) / 2)) < 1e-10
        assert 1 - 1e-12 <= smax < (1 + np.sqrt(5)) / 2
    # c = 1 cases: first step from A_0 = I/lambda with u = k_hat
    r = orc.forward_trace(q[:1], k[:1], v[:1], lam, flags=0)
    J = np.eye(dk) - np.outer(r.trace["alpha"][0], r.trace["khat"][0])
    assert abs(np.linalg.norm(J, 2) - 1) < 1e-12


def pin_paper_constants(orc, golden):
    """Printed values: lambda_0 = 0.1 gives A_0 = 10 I (Section 3.2) and ||A_0||_F ~ 56 at
    d_h = 32 (Section 6.2); eps = 1e-4."""
    lam, dh = golden["lambda0"], int(golden["d_h"])
    z = np.zeros((1, 1, 0, dh))
    r = orc.forward(z, z, z, lam, in_dtype=2)
    assert np.abs(r.A_T[0, 0] - golden["A0_diag"] * np.eye(dh)).max() < 1e-12
    assert abs(np.linalg.norm(r.A_T[0, 0]) - golden["A0_fro_approx"]) < 1.0   # printed as "~56"
    assert np.all(r.S_T == 0) and np.all(r.z_T == 0)


# --------------------------------------------------------------------------
# periodic identity refresh (Algorithm 1; Section 5.3: every 20 steps, + 1e-3 I)
# --------------------------------------------------------------------------
def pin_refresh_closed_form_with_zero_u(orc):
    """u = 0 leaves only the refresh: A_T = A_0 + (number of refresh steps) * eta * I, counted on
    the 1-based global position (carried step offset), and S still follows the normalised
    delta rule because A stays a multiple of I."""
    dk, dv, T, lam, eta, period = 5, 4, 47, 0.1, 1e-3, 20
    q, k, v, g = _rand(201, T, dk, dv)
    for off in (0, 7, 19, 33):
        r = orc.forward_trace(q, k, v, lam, u=np.zeros((T, dk)), flags=IDENT, refresh=(period, eta, off))
        n_ref = (off + T) // period - off // period
        assert np.abs(r.A_T - (1 / lam + n_ref * eta) * np.eye(dk)).max() < 1e-12
        for t in range(T):
            n_t = (off + t + 1) // period - off // period
            assert np.abs(r.trace["A"][t] - (1 / lam + n_t * eta) * np.eye(dk)).max() < 1e-12
        S = np.zeros((dv, dk))
        for t in range(T):
            kh = k[t] / np.linalg.norm(k[t])
            S = S + np.outer(v[t] - S @ kh, kh)
        assert np.abs(r.S_T - S).max() < 1e-12
    # a period longer than the sequence, or period 0, changes nothing
    base = orc.forward_trace(q, k, v, lam, flags=0)
    for rf in ((T + 1, eta, 0), (0, eta, 0), None):
        r = orc.forward_trace(q, k, v, lam, flags=0, refresh=rf)
        assert np.array_equal(r.out, base.out) and np.array_equal(r.A_T, base.A_T)


def pin_refresh_step_by_step_brute_force(orc):
    """A_t = (A_{t-1}^{-1} + u u^T)^{-1}, plus eta*I on refresh steps, with numpy inverses;
    the write direction uses the refreshed A_t (the refresh sits before it in Algorithm 1)."""
    dk, T, lam, eta, period = 6, 45, 0.2, 1e-3, 20
    q, k, v, g = _rand(211, T, dk, dk)
    for uu in (None, _unit(g.standard_normal((T, dk)))):
        r = orc.forward_trace(q, k, v, lam, u=uu, flags=0, refresh=(period, eta, 0))
        kh = _khat(k, 0)
        used = kh if uu is None else uu
        A = np.eye(dk) / lam
        for t in range(T):
            A = np.linalg.inv(np.linalg.inv(A) + np.outer(used[t], used[t]))
            if (t + 1) % period == 0:
                A = A + eta * np.eye(dk)
            assert np.abs(r.trace["A"][t] - A).max() < 1e-10 * np.abs(A).max(), t
            a = A @ kh[t]
            assert np.abs(r.trace["alpha"][t] - a / np.linalg.norm(a)).max() < 1e-10, t


def pin_refresh_state_carry(orc):
    """Split invariance needs the step offset to be carried along with (S, A, z)."""
    B, H, T, dk, dv, lam = 1, 2, 53, 5, 4, 0.1
    g = np.random.default_rng(221)
    q = g.standard_normal((B, H, T, dk)); k = g.standard_normal((B, H, T, dk))
    v = g.standard_normal((B, H, T, dv))
    full = orc.forward(q, k, v, lam, in_dtype=2, refresh=(20, 1e-3, 0))
    for T1 in (13, 20, 40):
        a = orc.forward(q[:, :, :T1], k[:, :, :T1], v[:, :, :T1], lam, in_dtype=2, refresh=(20, 1e-3, 0))
        b = orc.forward(q[:, :, T1:], k[:, :, T1:], v[:, :, T1:], lam, in_dtype=2, S0=a.S_T, A0=a.A_T,
                        z0=a.z_T, refresh=(20, 1e-3, T1))
        assert np.abs(np.concatenate([a.out, b.out], axis=2) - full.out).max() < 1e-12
        assert np.abs(b.A_T - full.A_T).max() < 1e-12 and np.abs(b.S_T - full.S_T).max() < 1e-12
    wrong = orc.forward(q[:, :, 13:], k[:, :, 13:], v[:, :, 13:], lam, in_dtype=2, refresh=(20, 1e-3, 0))
    assert np.abs(wrong.A_T - full.A_T).max() > 1e-6      # offset matters


def pin_segments_compose_through_a_transfer_scan(orc):
    """The facts the sequence-parallel GPU path rests on, checked on the oracle alone.  Cut a
    sequence in segments.  (i) A before a segment is the brute-force inverse of
    lambda I + sum of u u^T over the earlier tokens (Eq. "penalty").  (ii) With that A and the
    running key sum carried in, the segment scanned from S = 0 gives G and readouts o0_t; the
    same segment with v = 0 from S = I gives P and w_t; then S_end = S_start P + G and
    o_t = o0_t + S_start w_t (Section 3.4's composition with the map acting on the right)."""
    dk, T, lam = 7, 48, 0.3
    for flags in (0, IDENT):
        for with_u in (False, True):
            q, k, v, g = _rand(131 + flags, T, dk, dk)
            u = _unit(g.standard_normal((T, dk))) / np.sqrt(dk) if with_u else None
            S0 = 0.4 * g.standard_normal((dk, dk))
            z0 = g.uniform(0.0, 1.0, dk)
            full = orc.forward_trace(q, k, v, lam, u=u, S0=S0, z0=z0, flags=flags)
            uu = u if with_u else _khat(k, flags)
            kf = k if flags & IDENT else _phi(k)
            S_start = S0
            for a, b in ((0, 16), (16, 32), (32, 48)):
                A_start = np.linalg.inv(lam * np.eye(dk) + uu[:a].T @ uu[:a])
                z_start = z0 if flags & IDENT else z0 + kf[:a].sum(axis=0)
                sl = lambda x: None if x is None else np.ascontiguousarray(x[a:b])
                seg = orc.forward_trace(sl(q), sl(k), sl(v), lam, u=sl(u), A0=A_start, z0=z_start,
                                        flags=flags)
                tr = orc.forward_trace(sl(q), sl(k), np.zeros((b - a, dk)), lam, u=sl(u), S0=np.eye(dk),
                                       A0=A_start, z0=z_start, flags=flags)
                o = np.reshape(seg.out, (b - a, dk)) + np.reshape(tr.out, (b - a, dk)) @ S_start.T
                assert np.abs(o - np.reshape(full.out, (T, dk))[a:b]).max() < 1e-9
                S_start = S_start @ np.reshape(tr.S_T, (dk, dk)) + np.reshape(seg.S_T, (dk, dk))
            assert np.abs(S_start - np.reshape(full.S_T, (dk, dk))).max() < 1e-9
            assert np.abs(np.reshape(seg.A_T, (dk, dk)) - np.reshape(full.A_T, (dk, dk))).max() < 1e-9


# --------------------------------------------------------------------------
# Comparison mode: additive linear attention (Section 2, Eq. "linear-attn")
# --------------------------------------------------------------------------
LINATT = 2  # oracle.LINEAR_ATTENTION


def pin_linear_attention_is_a_direct_sum(orc):
    """o_t = sum_{s<=t} v_s (phi(k_s).phi(q_t)) / sum_{s<=t} phi(k_s).phi(q_t), S_T = sum v_s phi(k_s)^T,
    z_T = sum phi(k_s): written as plain double sums; A is passed through; carried states add on."""
    for dk, dv, T, seed in [(3, 2, 7, 1), (8, 8, 40, 2), (16, 5, 33, 3)]:
        q, k, v, g = _rand(seed, T, dk, dv)
        fk, fq = _phi(k), _phi(q)
        A0 = np.eye(dk) * 3.0 + 0.1
        r = orc.forward_trace(q, k, v, 0.7, flags=LINATT, A0=A0)
        for t in range(T):
            num = sum(v[s] * (fk[s] @ fq[t]) for s in range(t + 1))
            den = sum(fk[s] @ fq[t] for s in range(t + 1))
            assert np.abs(r.out[t] - num / den).max() < 1e-10 * max(1.0, np.abs(num / den).max()), (dk, t)
        assert np.abs(r.S_T - sum(np.outer(v[s], fk[s]) for s in range(T))).max() < 1e-10
        assert np.abs(r.z_T - fk.sum(axis=0)).max() < 1e-10
        assert np.array_equal(r.A_T, A0)                      # no penalty matrix in this mode
        # carried S0, z0 simply add to the sums; u is ignored
        S0, z0 = g.standard_normal((dv, dk)), np.abs(g.standard_normal(dk))
        r2 = orc.forward_trace(q, k, v, 0.7, flags=LINATT, S0=S0, z0=z0, u=g.standard_normal((T, dk)))
        t = T - 1
        num = S0 @ fq[t] + sum(v[s] * (fk[s] @ fq[t]) for s in range(T))
        den = z0 @ fq[t] + sum(fk[s] @ fq[t] for s in range(T))
        assert np.abs(r2.out[t] - num / den).max() < 1e-10 * max(1.0, np.abs(num / den).max())
        # with the identity map: S_T = sum v_s k_s^T and o_t = S_t q_t (no normaliser)
        r3 = orc.forward_trace(q, k, v, 0.7, flags=LINATT | IDENT)
        assert np.abs(r3.S_T - v.T @ k).max() < 1e-10
        assert np.abs(r3.out[T - 1] - (v.T @ k) @ q[T - 1]).max() < 1e-9


def pin_linear_attention_state_grows_where_vla_stays_bounded(orc):
    """Section 2's point about the additive update against Proposition 1: on the same random
    inputs ||S_t||_F of linear attention keeps growing (like sqrt(t) for zero-mean values; O(t) is
    the paper's bound), while the residual update's levels off far below it."""
    dk = dv = 16
    T = 600
    q, k, v, _ = _rand(11, T, dk, dv)
    la = orc.forward_trace(q, k, v, 0.1, flags=LINATT)
    vl = orc.forward_trace(q, k, v, 0.1)
    nla = np.linalg.norm(la.trace["S"].reshape(T, -1), axis=1)
    nvl = np.linalg.norm(vl.trace["S"].reshape(T, -1), axis=1)
    assert nla[-1] > 1.3 * nla[T // 2 - 1] > 1.3 * 1.3 * nla[T // 4 - 1]    # still growing
    assert nvl[T // 2:].max() < 1.5 * nvl[T // 4:T // 2].max()                # levelled off
    assert nla[-1] > 10 * nvl[-1]


PINS = [pin_A_is_brute_force_inverse, pin_A_invariants, pin_delta_value,
        pin_alpha_from_post_update_A, pin_first_step_closed_form,
        pin_orthonormal_keys_exact_recall, pin_repeated_key,
        pin_zero_u_is_normalised_delta_rule, pin_associative_composition,
        pin_proposition_1, pin_readout, pin_feature_map_values, pin_eps_guards,
        pin_state_carry, pin_units_layout_threads_dtypes, pin_jacobian_spectrum,
        pin_refresh_closed_form_with_zero_u, pin_refresh_step_by_step_brute_force,
        pin_refresh_state_carry, pin_segments_compose_through_a_transfer_scan,
        pin_linear_attention_is_a_direct_sum, pin_linear_attention_state_grows_where_vla_stays_bounded]
