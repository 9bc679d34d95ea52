"""Pins of the make_u oracle (u = scale * L2norm(W_u k), Algorithm 1) against what the
mathematics fixes, none of them a second copy of its formula: special cases that reduce to a
library norm, brute-force loops on tiny inputs, invariances."""
import math

import numpy as np
import pytest

import importlib.util
import os
import types

from oracle import make_u as ORACLE


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def pin_identity_projection_is_the_normalised_key(O):
    k = _rand((2, 3, 5, 8), 0).astype(np.float32)
    W = np.stack([np.eye(8)] * 3)
    u = O.make_u(k, W, scale=1.0)
    want = k.astype(np.float64) / np.linalg.norm(k.astype(np.float64), axis=-1, keepdims=True)
    np.testing.assert_allclose(u, want, rtol=1e-14, atol=0)


def pin_brute_force_per_head_and_orientation(O):
    """y_c = sum_j W[h][c][j] k_j with the head's own matrix, written as loops; a transposed or
    head-shared W fails."""
    B, H, T, d = 2, 3, 4, 5
    k = _rand((B, H, T, d), 1).astype(np.float32)
    W = _rand((H, d, d), 2)
    u = O.make_u(k, W, scale=0.37, eps=1e-4)
    for b in range(B):
        for h in range(H):
            for t in range(T):
                y = [sum(W[h][c][j] * float(k[b, h, t, j]) for j in range(d)) for c in range(d)]
                n = math.sqrt(sum(x * x for x in y))
                for c in range(d):
                    assert abs(u[b, h, t, c] - 0.37 * y[c] / n) <= 1e-14


def pin_norm_scale_and_invariances(O):
    k = _rand((1, 2, 7, 16), 3).astype(np.float32)
    W = _rand((2, 16, 16), 4)
    s = 16 ** -0.5
    u = O.make_u(k, W, scale=s)
    np.testing.assert_allclose(np.linalg.norm(u, axis=-1), s, rtol=1e-14)
    # positive rescaling of the keys or of the projection changes nothing; a sign flip flips u
    np.testing.assert_allclose(O.make_u(4.0 * k, W, scale=s), u, rtol=1e-13)
    np.testing.assert_allclose(O.make_u(k, 0.25 * W, scale=s), u, rtol=1e-13)
    np.testing.assert_allclose(O.make_u(k, -W, scale=s), -u, rtol=1e-13)


def pin_rotation_keeps_the_key_norm(O):
    """An orthogonal (non-symmetric) W: u = scale * Q k / ||k||."""
    q, _ = np.linalg.qr(_rand((6, 6), 5))
    assert np.abs(q - q.T).max() > 0.1
    k = _rand((1, 1, 9, 6), 6).astype(np.float32)
    u = O.make_u(k, q[None], scale=1.0)
    kk = k.astype(np.float64)[0, 0]
    want = np.stack([q.dot(kk[t]) / np.linalg.norm(kk[t]) for t in range(9)])
    np.testing.assert_allclose(u[0, 0], want, rtol=1e-12, atol=1e-15)


def pin_zero_key_and_guard(O):
    k = np.zeros((1, 1, 2, 4), dtype=np.float32)
    k[0, 0, 1] = [1e-7, 0, 0, 0]
    u = O.make_u(k, np.eye(4)[None], scale=1.0, eps=1e-4)
    assert np.all(u[0, 0, 0] == 0.0)
    np.testing.assert_allclose(u[0, 0, 1], [1e-3, 0, 0, 0], rtol=1e-6)   # y / eps below the guard


def pin_bf16_keys_are_widened_exactly(O):
    vals = np.array([1.0, -2.5, 0.15625, 3.0e-3], dtype=np.float32)
    bits = (vals.view(np.uint32) >> 16).astype(np.uint16)          # these values are bf16-exact or truncated
    back = O.widen(bits, O.BF16)
    np.testing.assert_array_equal(back, (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64))
    assert back[0] == 1.0 and back[1] == -2.5 and back[2] == 0.15625
    k = bits.reshape(1, 1, 1, 4)
    u = O.make_u(k, np.eye(4)[None], scale=1.0, in_dtype=O.BF16)
    np.testing.assert_allclose(u[0, 0, 0], back / np.linalg.norm(back), rtol=1e-14)


PINS = [pin_identity_projection_is_the_normalised_key, pin_brute_force_per_head_and_orientation, pin_norm_scale_and_invariances, pin_rotation_keeps_the_key_norm, pin_zero_key_and_guard, pin_bf16_keys_are_widened_exactly]


@pytest.mark.parametrize("pin", PINS, ids=lambda f: f.__name__)
def test_pin(pin):
    pin(ORACLE)


# ---- planted mistakes: each must trip at least one pin
MUTANTS = [
    ("transposed projection", "y = kk[b, h] @ W[h].T", "y = kk[b, h] @ W[h]"),
    ("head-shared projection", "y = kk[b, h] @ W[h].T", "y = kk[b, h] @ W[0].T"),
    ("scale dropped", "u[b, h] = scale * y / np.maximum(nrm, eps)[:, None]", "u[b, h] = y / np.maximum(nrm, eps)[:, None]"),
    ("no normalisation", "u[b, h] = scale * y / np.maximum(nrm, eps)[:, None]", "u[b, h] = scale * y"),
    ("squared norm", "nrm = np.sqrt((y * y).sum(axis=1))", "nrm = (y * y).sum(axis=1)"),
    ("norm over tokens", "nrm = np.sqrt((y * y).sum(axis=1))", "nrm = np.sqrt((y * y).sum(axis=0))[None, :].repeat(y.shape[0], 0)[:, 0]"),
    ("guard added instead of clamped", "np.maximum(nrm, eps)", "(nrm + eps)"),
    ("bf16 widened as integers", "return bits.view(np.float32).astype(np.float64)", "return bits.astype(np.float64)"),
]


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistakes_trip_a_pin(name, old, new):
    src = open(os.path.join(os.path.dirname(ORACLE.__file__), "make_u.py")).read()
    assert src.count(old) >= 1, "mutation site not found: " + name
    mod = types.ModuleType("make_u_mutant")
    exec(compile(src.replace(old, new), "make_u_mutant", "exec"), mod.__dict__)
    tripped = []
    for pin in PINS:
        try:
            pin(mod)
        except Exception:                      # a failed assertion or a numerical blow-up both count
            tripped.append(pin.__name__)
    assert tripped, "no pin notices: " + name
