"""Pins for the backward oracle (oracle/vla_oracle_bwd.c): it is hand-written reverse-mode
differentiation, so what fixes it is the forward oracle itself -- central finite differences of
``vla_oracle_forward`` for a random linear functional of everything the forward returns, for
every input, in every mode -- plus linearity in the incoming gradients and a one-token closed
form.  A handful of planted mistakes in a copy of the C file must each trip the pins."""
import os
import re
import subprocess
import sys

import numpy as np
import pytest

import oracle

IDENT = oracle.IDENTITY_MAP
HERE = os.path.dirname(os.path.abspath(__file__))


def _case(seed, B, H, T, d, with_u, with_state):
    g = np.random.default_rng(seed)
    x = {"q": g.standard_normal((B, H, T, d)), "k": g.standard_normal((B, H, T, d)),
         "v": g.standard_normal((B, H, T, d))}
    if with_u:
        u = g.standard_normal((B, H, T, d))
        x["u"] = 0.8 * u / np.linalg.norm(u, axis=-1, keepdims=True)
    if with_state:
        x["S0"] = 0.5 * g.standard_normal((B, H, d, d))
        h = 0.4 * g.standard_normal((B, H, d, d))
        x["A0"] = h @ np.swapaxes(h, -1, -2) + 0.7 * np.eye(d)
        x["z0"] = g.uniform(0.2, 1.5, (B, H, d))
    w = {"o": g.standard_normal((B, H, T, d)), "S": g.standard_normal((B, H, d, d)),
         "A": g.standard_normal((B, H, d, d)), "z": g.standard_normal((B, H, d))}
    return x, w


def _loss(x, w, lam, flags, refresh):
    r = oracle.forward(x["q"], x["k"], x["v"], lam, u=x.get("u"), in_dtype=oracle.F64, S0=x.get("S0"),
                       A0=x.get("A0"), z0=x.get("z0"), flags=flags, refresh=refresh)
    return float((w["o"] * r.out).sum() + (w["S"] * r.S_T).sum() + (w["A"] * r.A_T).sum() +
                 (w["z"] * r.z_T).sum())


def _grads(bwd, x, w, lam, flags, refresh):
    g = bwd.backward(x["q"], x["k"], x["v"], lam, w["o"], u=x.get("u"), S0=x.get("S0"), A0=x.get("A0"),
                     z0=x.get("z0"), dS_T=w["S"], dA_T=w["A"], dz_T=w["z"], flags=flags, refresh=refresh)
    return {"q": g.dq, "k": g.dk, "v": g.dv, "u": g.du, "S0": g.dS0, "A0": g.dA0, "z0": g.dz0}


def finite_difference_mismatch(bwd, seed, T, d, flags, with_u, with_state, refresh, lam=0.3, h=1e-6):
    """Largest |analytic - central difference| / scale over every coordinate of every input."""
    x, w = _case(seed, 1, 2, T, d, with_u, with_state)
    an = _grads(bwd, x, w, lam, flags, refresh)
    worst = 0.0
    for name in x:
        num = np.zeros_like(x[name])
        it = np.nditer(x[name], flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            keep = x[name][idx]
            x[name][idx] = keep + h
            lp = _loss(x, w, lam, flags, refresh)
            x[name][idx] = keep - h
            lm = _loss(x, w, lam, flags, refresh)
            x[name][idx] = keep
            num[idx] = (lp - lm) / (2 * h)
        scale = max(1.0, np.abs(num).max())
        worst = max(worst, float(np.abs(an[name] - num).max() / scale))
    return worst


CASES = [  # (T, d, flags, explicit u, carried state, refresh)
    (5, 3, 0, False, False, None),
    (5, 3, IDENT, False, False, None),
    (6, 4, 0, True, True, None),
    (6, 4, IDENT, True, True, None),
    (7, 3, 0, False, True, (3, 0.05, 1)),
    (7, 3, 0, True, True, (2, 0.1, 0)),
    (1, 4, 0, False, True, None),
]


def pins_hold(bwd) -> str:
    """Returns the name of the first pin that fails for this build, or '' when all hold."""
    for n, (T, d, flags, with_u, with_state, refresh) in enumerate(CASES):
        if finite_difference_mismatch(bwd, 300 + n, T, d, flags, with_u, with_state, refresh) > 2e-6:
            return "finite differences, case %d" % n
    # linear in the incoming gradients
    x, w = _case(7, 1, 1, 6, 4, True, True)
    w2 = {k2: 2.5 * v for k2, v in w.items()}
    g1, g2 = _grads(bwd, x, w, 0.5, 0, None), _grads(bwd, x, w2, 0.5, 0, None)
    for name in g1:
        if np.abs(g2[name] - 2.5 * g1[name]).max() > 1e-10 * max(1.0, np.abs(g1[name]).max()):
            return "linearity"
    # one token from S0 = 0, identity map, only o weighted: o = v (alpha.q), alpha = k_hat
    # (A_0 = I/lambda), so dL/dv = w_o (k_hat.q)
    g = np.random.default_rng(5)
    q, k, v = (g.standard_normal((1, 1, 1, 5)) for _ in range(3))
    wo = g.standard_normal((1, 1, 1, 5))
    r = bwd.backward(q, k, v, 0.7, wo, flags=IDENT)
    kh = k[0, 0, 0] / np.linalg.norm(k[0, 0, 0])
    if np.abs(r.dv[0, 0, 0] - wo[0, 0, 0] * (kh @ q[0, 0, 0])).max() > 1e-12:
        return "one-token closed form"
    return ""


def test_backward_oracle_matches_finite_differences_of_the_forward_oracle():
    assert pins_hold(oracle.load_bwd()) == ""


MUTANTS = [
    ("dden sign", "-odo / (den[t] * den[t])", "odo / (den[t] * den[t])"),
    ("readout gradient uses the reverted S", "dqf[j] = s + dden * zk[j];", "dqf[j] = s;"),
    ("alpha normalisation term dropped", "da[j] = (dal[j] - al[j] * ad) / na[t];", "da[j] = dal[j] / na[t];"),
    ("dz misses the transpose", "(GA[(size_t)i * dk + j] + GA[(size_t)j * dk + i]) * zt[j]",
     "(2.0 * GA[(size_t)i * dk + j]) * zt[j]"),
    ("ddelta dropped", "ddelta /= delta[t] * delta[t];", "ddelta = 0.0;"),
    ("residual gradient before undoing the S update",
     "S[(size_t)i * dk + j] -= et[i] * al[j];   /* back to S */", ";"),
    ("key normalisation term dropped", "dkf[j] += (dkh[j] - kh[j] * kd) / nk[t];", "dkf[j] += dkh[j] / nk[t];"),
    ("feature-map derivative", "static double dphi(double x) { return x > 0.0 ? 1.0 : exp(x); }",
     "static double dphi(double x) { return x > 0.0 ? 1.0 : exp(x) + 1.0; }"),
    ("key-sum gradient not carried", "for (int j = 0; j < dk; ++j) gz[j] += dden * qft[j];",
     "for (int j = 0; j < dk; ++j) gz[j] = dden * qft[j];"),
    ("refresh not undone", "for (int i = 0; i < dk; ++i) A[(size_t)i * dk + i] -= J->rf->eta;", ";"),
]


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_in_a_copy_is_noticed(tmp_path, name, old, new):
    src = open(os.path.join(os.path.dirname(HERE), "oracle", "vla_oracle_bwd.c")).read()
    assert src.count(old) == 1, "mutant pattern must match exactly once: %r" % old
    c = tmp_path / "mutant_bwd.c"
    c.write_text(src.replace(old, new))
    so = str(tmp_path / "libmutant_bwd.so")
    oracle.build_bwd(force=True, src=str(c), out=so)
    code = ("import sys; sys.path[:0] = [%r, %r]; import oracle, test_oracle_bwd_pins as m; "
            "print('TRIPPED', repr(m.pins_hold(oracle.OracleBwdLib(%r))))" % (HERE, os.path.dirname(HERE), so))
    res = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=600)
    if res.returncode != 0:
        return                      # the mutant crashed: noticed
    tripped = res.stdout.strip().split("TRIPPED")[-1].strip()
    assert tripped not in ("''", '""'), "no pin notices the planted mistake %r" % name
