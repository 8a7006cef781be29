"""Do the pins bite?  Each case plants ONE plausible mistake in a copy of the CPU checker's source
(a dropped term, a wrong sign or index, a transposed operand, a wrong boundary), runs the pins of
tests/test_oracle_pins.py against the mutated copy and requires that at least one of them fails.
Everything here runs on the CPU; the CUDA library is not involved."""
import inspect
import types

import numpy as np
import pytest

from oracle import gswa_oracle as orc

import test_oracle_pins as pins

SRC = inspect.getsource(orc)

# (name, text in the checker's source, replacement)
MUTATIONS = [
    ("shift-direction", "np.roll(t, shift=(-s, -s), axis=(1, 2)) if s else t", "np.roll(t, shift=(s, s), axis=(1, 2)) if s else t"),
    ("shift-one-axis-only", "np.roll(t, shift=(-s, -s), axis=(1, 2)) if s else t", "np.roll(t, shift=(-s, 0), axis=(1, 2)) if s else t"),
    ("region-boundary", "r[n - M:n - s] = 1", "r[n - M:n - s - 1] = 1"),
    ("regions-merged", "r[n - s:] = 2", "r[n - s:] = 1"),
    ("mask-finite", "np.where(same, 0.0, -np.inf)", "np.where(same, 0.0, -100.0)"),
    ("mask-dropped", "S = (S.reshape(B, nW, gh, N, N) + mask[None, :, None]).reshape(B * nW, gh, N, N)", "pass"),
    ("rel-transposed", "rel = (a[:, None] - a[None, :] + M - 1) * (2 * M - 1) + (c[:, None] - c[None, :] + M - 1)",
     "rel = (a[None, :] - a[:, None] + M - 1) * (2 * M - 1) + (c[None, :] - c[:, None] + M - 1)"),
    ("rel-row-col-swapped", "rel = (a[:, None] - a[None, :] + M - 1) * (2 * M - 1) + (c[:, None] - c[None, :] + M - 1)",
     "rel = (c[:, None] - c[None, :] + M - 1) * (2 * M - 1) + (a[:, None] - a[None, :] + M - 1)"),
    ("scale-dropped", "scale = float(dq) ** -0.5", "scale = 1.0"),
    ("softmax-over-queries", "Smax = S.max(axis=-1, keepdims=True)\n        E = np.exp(S - Smax)\n        P = E / E.sum(axis=-1, keepdims=True)",
     "Smax = S.max(axis=-2, keepdims=True)\n        E = np.exp(S - Smax)\n        P = E / E.sum(axis=-2, keepdims=True)"),
    ("bias-head-offset", "S = S + table[rel][:, :, h0:h0 + gh].transpose(2, 0, 1)[None]", "S = S + table[rel][:, :, 0:gh].transpose(2, 0, 1)[None]"),
    ("partition-transposed", "t = t.reshape(B, H // M, M, W // M, M, c).transpose(0, 1, 3, 2, 4, 5)\n    return t.reshape(B * (H // M) * (W // M), M * M, c)",
     "t = t.reshape(B, H // M, M, W // M, M, c).transpose(0, 1, 3, 4, 2, 5)\n    return t.reshape(B * (H // M) * (W // M), M * M, c)"),
    ("proj-not-transposed", "y = A @ w_proj.T + b_proj                                               # W^P of Eq. 7", "y = A @ w_proj + b_proj"),
    ("bwd-softmax-jacobian-term", "dS = P * (dP - (P * dP).sum(axis=-1, keepdims=True))", "dS = P * dP"),
    ("bwd-dq-scale", "dqkv = np.concatenate([dq * scale, dk, dv], axis=-1)", "dqkv = np.concatenate([dq, dk, dv], axis=-1)"),
    ("bwd-dk-operands", 'dkw = np.einsum("nhpq,nphd->nqhd", dS, qw)', 'dkw = np.einsum("nhpq,nqhd->nphd", dS, qw)'),
    ("bwd-dv-uses-dS", 'dvw = np.einsum("nhpq,nphd->nqhd", P, dO)', 'dvw = np.einsum("nhpq,nphd->nqhd", dS if False else P.transpose(0, 1, 3, 2), dO)'),
    ("bwd-dtable-head", "np.add.at(dtable[:, h0 + hh], rel.ravel(), dSh[hh].ravel())", "np.add.at(dtable[:, hh], rel.ravel(), dSh[hh].ravel())"),
    ("bwd-dtable-transposed", "np.add.at(dtable[:, h0 + hh], rel.ravel(), dSh[hh].ravel())", "np.add.at(dtable[:, h0 + hh], rel.T.ravel(), dSh[hh].ravel())"),
    ("bwd-dwproj-transposed", "dw_proj = dy2.T @ A.reshape(-1, A.shape[-1])", "dw_proj = A.reshape(-1, A.shape[-1]).T @ dy2"),
    ("bwd-reverse-shift-dropped", "dst[..., sl] = reverse_shift(window_reverse(src.reshape(-1, N, gh * wd), M, B, H, W), s)",
     "dst[..., sl] = window_reverse(src.reshape(-1, N, gh * wd), M, B, H, W)"),
    ("bwd-dx-weight-transposed", "dx = (dqkv @ w_qkv).reshape(B, H, W, C)", "dx = (dqkv @ w_qkv[:, ::-1]).reshape(B, H, W, C)"),
]


def _pin_calls():
    """The pins, with the parameters pytest would give them (a subset of the parametrisations keeps this quick)."""
    calls = []
    for H, W, M in [(8, 16, 4), (6, 6, 3)]:
        calls.append((pins.test_partition_reverse_and_shift_unshift_are_identities, (H, W, M)))
        calls.append((pins.test_index_maps_match_roll_and_partition_of_a_token_counter, (H, W, M)))
        calls.append((pins.test_three_forms_of_the_pair_predicate_agree, (H, W, M)))
    calls.append((pins.test_procedural_forward_equals_bruteforce_global_attention, (8, 8, 4, (0, 1))))
    calls.append((pins.test_procedural_forward_equals_bruteforce_global_attention, (6, 6, 3, (1, 2))))
    calls.append((pins.test_shift_zero_is_textbook_window_attention, ()))
    calls.append((pins.test_masked_weights_are_exactly_zero_and_rows_sum_to_one, ()))
    calls.append((pins.test_closed_form_when_queries_keys_and_table_vanish, ()))
    calls.append((pins.test_batch_items_are_independent, ()))
    calls.append((pins.test_gradients_match_central_finite_differences, (8, 12, 4, (2, 1), (3, 1))))
    calls.append((pins.test_gradient_invariants, ()))
    return calls


def _mutated_module(old: str, new: str):
    assert SRC.count(old) >= 1, "mutation target not found in the checker's source: %r" % old
    mod = types.ModuleType("gswa_oracle_mutant")
    exec(compile(SRC.replace(old, new), "gswa_oracle_mutant", "exec"), mod.__dict__)
    return mod


def _first_failure(monkeypatch, mod):
    monkeypatch.setattr(pins, "orc", mod)
    for fn, args in _pin_calls():
        try:
            with np.errstate(all="ignore"):
                fn(*args)
        except AssertionError:
            return fn.__name__
        except (ValueError, IndexError, FloatingPointError):
            return fn.__name__ + " (raised)"
    return None


def test_unmutated_copy_passes_every_pin(monkeypatch):
    mod = _mutated_module("F64 = np.float64", "F64 = np.float64 ")
    assert _first_failure(monkeypatch, mod) is None


@pytest.mark.parametrize("name,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_is_caught(monkeypatch, name, old, new):
    mod = _mutated_module(old, new)
    assert _first_failure(monkeypatch, mod) is not None, "no pin noticed the planted mistake '%s'" % name
