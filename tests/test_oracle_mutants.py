"""The pins have teeth: each plausible mistake, planted in a COPY of the oracle's C
file (on the CPU, in a temp directory), must trip at least one pin.  The committed
oracle itself is never modified."""
import os
import subprocess
import sys

import pytest

import oracle
from oracle_pins import PINS, pin_paper_constants
from test_oracle_pins import read_golden

SRC = os.path.join(os.path.dirname(oracle.__file__), "vla_oracle.c")

# (name, text in the oracle, replacement)
MUTANTS = [
    ("sm_sign", "-= gain[i] * gain[j] / delta;", "+= gain[i] * gain[j] / delta;"),
    ("sm_no_division", "-= gain[i] * gain[j] / delta;", "-= gain[i] * gain[j];"),
    ("delta_drops_one", "double delta = 1.0 + dot(pen, gain, dk);", "double delta = dot(pen, gain, dk);"),
    ("delta_wrong_dot", "double delta = 1.0 + dot(pen, gain, dk);", "double delta = 1.0 + dot(gain, gain, dk);"),
    ("z_uses_khat", "delta = inverse_penalty_step(A, pen, gain, dk, eps);",
     "delta = inverse_penalty_step(A, key_unit, gain, dk, eps);"),
    ("u_ignored", "pen[j] = u_in ? load_elem(u_in, row_k + j, dtype) : key_unit[j];", "pen[j] = key_unit[j];"),
    ("alpha_from_pre_update_A", "unit_write_direction(A, key_unit, write_dir, dk, eps);\n      residual_write",
     "for (int i = 0; i < dk; ++i) for (int j = 0; j < dk; ++j) A[(size_t)i * dk + j] += gain[i] * gain[j] / delta;\n"
     "      unit_write_direction(A, key_unit, write_dir, dk, eps);\n"
     "      for (int i = 0; i < dk; ++i) for (int j = 0; j < dk; ++j) A[(size_t)i * dk + j] -= gain[i] * gain[j] / delta;\n"
     "      residual_write"),
    ("alpha_not_normalised", "write_dir[i] /= guard;", "write_dir[i] /= 1.0;"),
    ("khat_not_normalised", "key_unit[j] = key_map[j] / guard;", "key_unit[j] = key_map[j];"),
    ("residual_sign", "- dot(S + (size_t)i * dk, key_unit, dk);", "+ dot(S + (size_t)i * dk, key_unit, dk);"),
    ("residual_no_prediction", "- dot(S + (size_t)i * dk, key_unit, dk);", ";"),
    ("write_along_khat", "S[(size_t)i * dk + j] += resid[i] * write_dir[j];", "S[(size_t)i * dk + j] += resid[i] * key_unit[j];"),
    ("write_sign", "S[(size_t)i * dk + j] += resid[i] * write_dir[j];", "S[(size_t)i * dk + j] -= resid[i] * write_dir[j];"),
    ("readout_pre_update_S", "double den = read_out(S, q, row_k,",
     "for (int i = 0; i < dv; ++i) for (int j = 0; j < dk; ++j) S[(size_t)i * dk + j] -= resid[i] * write_dir[j];\n"
     "    double den = read_out(S, q, row_k,"),
    ("readout_no_normaliser", "o[i] = dot(S + (size_t)i * dk, qry_map, dk) / den;", "o[i] = dot(S + (size_t)i * dk, qry_map, dk);"),
    ("den_excludes_current_token", "den = dot(key_sum, qry_map, dk);", "den = dot(key_sum, qry_map, dk) - dot(key_map, qry_map, dk);"),
    ("elu_without_plus_one", "return x > 0.0 ? x + 1.0 : exp(x);", "return x > 0.0 ? x : exp(x) - 1.0;"),
    ("phi_wrong_branch", "return x > 0.0 ? x + 1.0 : exp(x);", "return x > 0.0 ? x + 1.0 : 1.0 + x;"),
    ("q_not_mapped", "qry_map[j] = identity ? raw : phi(raw);", "qry_map[j] = raw;"),
    ("A0_is_lambda_I", "A[i * dk + i] = 1.0 / jb->lambda;", "A[i * dk + i] = jb->lambda;"),
    ("z0_ignored", "if (jb->z0) memcpy(zk,", "if (0) memcpy(zk,"),
    ("S0_ignored", "if (jb->S0) memcpy(S,", "if (0) memcpy(S,"),
    ("out_unit_stride", "jb->out + (size_t)n * T * dv, jb->tr, jb->rf);", "jb->out + (size_t)n * T * dk, jb->tr, jb->rf);"),
    ("bf16_shift", "[idx] << 16;", "[idx] << 15;"),
    ("refresh_wrong_step", "(rf->step_offset + t + 1) % rf->period == 0", "(rf->step_offset + t) % rf->period == 0"),
    ("refresh_ignores_offset", "(rf->step_offset + t + 1) % rf->period == 0", "(t + 1) % rf->period == 0"),
    ("refresh_sign", "A[(size_t)i * dk + i] += rf->eta;", "A[(size_t)i * dk + i] -= rf->eta;"),
    ("refresh_every_step", "rf->period > 0 && (rf->step_offset + t + 1) % rf->period == 0", "rf->period > 0"),
    ("eps_guard_missing", "double guard = len > eps ? len : eps;\n  for (int j = 0; j < dk; ++j) key_unit[j]",
     "double guard = len;\n  for (int j = 0; j < dk; ++j) key_unit[j]"),
    ("additive_normalises_key", "additive_write(S, v, row_v, dtype, key_map, resid, dk, dv);",
     "additive_write(S, v, row_v, dtype, key_unit, resid, dk, dv);"),
    ("additive_write_sign", "S[(size_t)i * dk + j] += resid[i] * key_map[j];", "S[(size_t)i * dk + j] -= resid[i] * key_map[j];"),
    ("additive_subtracts_prediction", "resid[i] = load_elem(v, row_v + i, dtype);\n    for",
     "resid[i] = load_elem(v, row_v + i, dtype) - dot(S + (size_t)i * dk, key_map, dk);\n    for"),
    ("additive_touches_A", "      for (int j = 0; j < dk; ++j) { pen[j] = 0.0; write_dir[j] = key_map[j]; }",
     "      for (int j = 0; j < dk; ++j) { pen[j] = 0.0; write_dir[j] = key_map[j]; }\n"
     "      inverse_penalty_step(A, key_unit, gain, dk, eps);"),
]


def _tripped_by(orc):
    for pin in PINS:
        try:
            pin(orc)
        except Exception:          # AssertionError, or a LinAlgError from a non-finite state
            return pin.__name__
    try:
        pin_paper_constants(orc, read_golden())
    except Exception:
        return "pin_paper_constants"
    return None


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_mutant_is_caught(tmp_path, name, old, new):
    text = open(SRC).read()
    assert text.count(old) == 1, "mutation site must match the oracle source exactly once: %r" % old
    c = tmp_path / "vla_oracle.c"
    c.write_text(text.replace(old, new))
    (tmp_path / "vla_oracle.h").write_text(open(SRC[:-2] + ".h").read())
    so = str(tmp_path / ("mut_%s.so" % name))
    subprocess.check_call(["gcc", "-std=c99", "-O2", "-fPIC", "-shared", "-w", "-o", so, str(c),
                           "-lm", "-lpthread"])
    # a child process, so that a mutant that corrupts memory cannot take pytest down
    here = os.path.dirname(os.path.abspath(__file__))
    code = ("import sys; sys.path[:0] = [%r, %r]; import oracle, test_oracle_mutants as m; "
            "print('CAUGHT_BY', m._tripped_by(oracle.OracleLib(%r)))" % (here, os.path.dirname(here), so))
    res = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=300)
    if res.returncode != 0:
        return                      # the mutant crashed: noticed
    caught = res.stdout.strip().split("CAUGHT_BY")[-1].strip()
    assert caught != "None", "no pin notices the planted mistake %r" % name
