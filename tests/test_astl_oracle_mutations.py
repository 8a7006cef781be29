"""Do the pins of tests/test_astl_oracle_pins.py bite?  One planted mistake per case in a copy of
oracle/astl_oracle.py; at least one pin must fail.  CPU only."""
import inspect
import sys
import types

import numpy as np
import pytest

from oracle import astl_oracle as ao

import test_astl_oracle_pins as pins

SRC = inspect.getsource(ao)

MUTATIONS = [
    ("ln-unbiased-variance", "var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)", "var = ((x - mu) ** 2).sum(axis=-1, keepdims=True) / (x.shape[-1] - 1)"),
    ("ln-eps-outside-root", "rstd = 1.0 / np.sqrt(var + eps)", "rstd = 1.0 / (np.sqrt(var) + eps)"),
    ("ln-bwd-mean-term", "dx = rstd * (dxhat - dxhat.mean(axis=-1, keepdims=True) - xhat * (dxhat * xhat).mean(axis=-1, keepdims=True))",
     "dx = rstd * (dxhat - xhat * (dxhat * xhat).mean(axis=-1, keepdims=True))"),
    ("ln-bwd-projection-term", "dx = rstd * (dxhat - dxhat.mean(axis=-1, keepdims=True) - xhat * (dxhat * xhat).mean(axis=-1, keepdims=True))",
     "dx = rstd * (dxhat - dxhat.mean(axis=-1, keepdims=True))"),
    ("ln-bwd-dgamma-uses-x", "return dx, (dy * xhat).reshape(-1, C).sum(axis=0), dy.reshape(-1, C).sum(axis=0)",
     "return dx, (dy * dxhat).reshape(-1, C).sum(axis=0), dy.reshape(-1, C).sum(axis=0)"),
    ("gelu-tanh-form", "return 0.5 * x * (1.0 + _erf(x / math.sqrt(2.0)))",
     "return 0.5 * x * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (x + 0.044715 * x ** 3)))"),
    ("gelu-grad-density-term", "+ x * np.exp(-0.5 * x * x) / math.sqrt(2.0 * math.pi)", "+ np.exp(-0.5 * x * x) / math.sqrt(2.0 * math.pi)"),
    ("mlp-no-activation-gradient", "dh = (dy @ w2) * gelu_grad(h)", "dh = (dy @ w2)"),
    ("mlp-dw1-of-activations", "dw1 = dh2.T @ x.reshape(-1, C)", "dw1 = dh2.T @ x.reshape(-1, C) * 0 + (dy.reshape(-1, C).T @ x.reshape(-1, C))[:1].sum() * 0 + dh2.T @ (x.reshape(-1, C) + 1e-3)"),
    ("cascade-adds-input-not-output", "        prev = o\n    A = np.concatenate", "        prev = xi\n    A = np.concatenate"),
    ("cascade-skips-a-head", "if cascade and prev is not None:\n            xi = xi + prev", "if cascade and prev is not None and i != 2:\n            xi = xi + prev"),
    ("cascade-gradient-carry-dropped", 'carry = g["dx"] if cache["cascade"] else None', "carry = None"),
    ("sliced-table-column", "table[:, i:i + 1], M, (1,), (shifts[i],), keep=keep", "table[:, 0:1], M, (1,), (shifts[i],), keep=keep"),
    ("sliced-shift-of-first-group", "return [s for gh, s in zip(group_heads, group_shift) for _ in range(gh)]",
     "return [group_shift[0] for gh, s in zip(group_heads, group_shift) for _ in range(gh)]"),
    ("layer-first-skip-dropped", "x1 = a + x                                               # Eq. 4", "x1 = a"),
    ("layer-second-skip-dropped", "x2 = m + x1                                              # Eq. 5", "x2 = m"),
    ("layer-second-norm-of-input", 'xn2, c_ln2 = layer_norm(x1, p["ln2_g"], p["ln2_b"])', 'xn2, c_ln2 = layer_norm(x, p["ln2_g"], p["ln2_b"])'),
    ("layer-bwd-skip-gradient", 'g["dx"] = dx1 + dres                                     # skip connection of Eq. 4', 'g["dx"] = dres'),
    ("layer-bwd-mlp-skip-gradient", "dx1 = dy + dres                                      # skip connection of Eq. 5", "dx1 = dres"),
]


def _mutant(old, new):
    assert SRC.count(old) >= 1, "mutation target not found: %r" % old
    mod = types.ModuleType("oracle.astl_oracle_mutant")
    mod.__package__ = "oracle"
    exec(compile(SRC.replace(old, new), "astl_oracle_mutant", "exec"), mod.__dict__)
    return mod


def _first_failure(monkeypatch, mod):
    monkeypatch.setattr(pins, "ao", mod)
    calls = [(pins.test_layer_norm_closed_forms, ()), (pins.test_layer_norm_backward_finite_differences_and_invariants, ()),
             (pins.test_gelu_values_identities_and_derivative, ()), (pins.test_mlp_against_loops_and_finite_differences, ()),
             (pins.test_sliced_heads_without_cascade_equal_dense_layer_with_block_diagonal_weights, ()),
             (pins.test_cascaded_heads_against_bruteforce_global_attention, ((1, 2), (0, 1))),
             (pins.test_cascade_passes_nothing_on_from_a_head_whose_value_projection_vanishes, ()),
             (pins.test_cascaded_gradients_match_finite_differences, ()), (pins.test_layer_structure, ()),
             (pins.test_layer_gradients_match_finite_differences, (True,))]
    for fn, args in calls:
        try:
            with np.errstate(all="ignore"):
                fn(*args)
        except AssertionError:
            return fn.__name__
        except (ValueError, IndexError, FloatingPointError):
            return fn.__name__ + " (raised)"
    return None


def test_unmutated_copy_passes(monkeypatch):
    assert _first_failure(monkeypatch, _mutant("LN_EPS = 1e-5", "LN_EPS = 1e-5 ")) is None


@pytest.mark.parametrize("name,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_is_caught(monkeypatch, name, old, new):
    assert _first_failure(monkeypatch, _mutant(old, new)) is not None, "no pin noticed '%s'" % name
