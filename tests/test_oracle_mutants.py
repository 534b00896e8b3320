"""The pins must be able to fail: each plausible mistake planted in a copy of the oracle (on the CPU)
is caught by at least one of them."""
import importlib.util
import os
import sys
import types

import pytest

import tests.test_oracle_pins as pins

SRC = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "oracle", "ulorl_oracle.py")

MUTANTS = {
    "entropy sign": ("ent[a:a + chunk] = -(p * lnp).sum(axis=1)", "ent[a:a + chunk] = (p * lnp).sum(axis=1)"),
    "kappa dropped from the logits": ("z = float(kappa) * (_f64(hidden[r]) @ W64.T)\n        m = z.max(axis=1)\n        lse_c",
                                      "z = (_f64(hidden[r]) @ W64.T)\n        m = z.max(axis=1)\n        lse_c"),
    "kappa dropped from the gradient": ("dz *= (float(kappa) * float(grad_loss) * g[r])[:, None]",
                                        "dz *= (float(grad_loss) * g[r])[:, None]"),
    "one-hot sign": ("dz[np.arange(r.shape[0]), targets[r]] += 1.0", "dz[np.arange(r.shape[0]), targets[r]] -= 1.0"),
    "dW uses the wrong operand": ("dW += dz.T @ h", "dW += dz.T @ (h * 0 + 1)"),
    "clip bounds swapped": ("c = min(max(r, 1.0 - eps_lo), 1.0 + eps_hi)\n            s = min(r * A, c * A)\n            keep",
                            "c = min(max(r, 1.0 - eps_hi), 1.0 + eps_lo)\n            s = min(r * A, c * A)\n            keep"),
    "max instead of min": ("s = min(r * A, c * A)\n            keep", "s = max(r * A, c * A)\n            keep"),
    "mask ignores the advantage sign": ("mpt = bool(A32 > 0) and bool(logp32[t] >= ln_tau)", "mpt = bool(logp32[t] >= ln_tau)"),
    "strict tau": ("bool(logp32[t] >= ln_tau)", "bool(logp32[t] > ln_tau)"),
    "gate not strict": ("gate = bool(gate_ent32[i] < sigma32)", "gate = bool(gate_ent32[i] <= sigma32)"),
    "normaliser counts unmasked tokens only": ("    loss = -loss_sum / N\n", "    loss = -loss_sum / max(1.0, float(np.count_nonzero((flags & FLAG_MASKED) == 0)))\n"),
    "clipped tokens keep their gradient": ("keep * (A * r * (0.0 if (hi or lo) else 1.0) - beta * dk)", "keep * (A * r - beta * dk)"),
    "ratio inverted": ("d32 = np.float32(logp32[t] - np.float32(old_logp[t]))", "d32 = np.float32(np.float32(old_logp[t]) - logp32[t])"),
    "masked tokens keep their gradient": ("g = -(1.0 / N) * keep * (A * r *", "g = -(1.0 / N) * (A * r *"),
    "KL term enters with the wrong sign": ("loss_sum += keep * (s - beta * kl[t]) * wlen", "loss_sum += keep * (s + beta * kl[t]) * wlen"),
    "KL gradient sign": ("dk = 1.0 - float(np.exp(u))", "dk = float(np.exp(u)) - 1.0"),
    "KL direction reversed": ("u = float(np.float64(np.float32(ref_logp[t])) - np.float64(logp32[t]))", "u = float(np.float64(logp32[t]) - np.float64(np.float32(ref_logp[t])))"),
    "KL term outside the mask": ("loss_sum += keep * (s - beta * kl[t]) * wlen", "loss_sum += (keep * s - beta * kl[t]) * wlen"),
    "KL estimate without its linear term": ("return np.exp(u) - u - 1.0", "return np.exp(u) - 1.0"),
    "sample std in the advantages": ("std = (var / G) ** 0.5", "std = (var / (G - 1)) ** 0.5"),
    "advantage sign": ("adv[a + j] = (grp[j] - mean) / std if std > 0 else 0.0", "adv[a + j] = (mean - grp[j]) / std if std > 0 else 0.0"),
    "group filter keeps all-correct groups": ("kept = 0 < n_correct < G", "kept = 0 < n_correct <= G"),
    "per-sample weight forgotten in the gradient": ("- beta * dk) * wlen + 0.0", "- beta * dk) + 0.0"),
    "per-sample weight uses T": ("1.0 / max(1.0, float(off[i + 1] - off[i]))", "1.0 / float(T)"),
    "per-sample mode divides by tokens": ("N = float(p.norm_seqs) if p.norm_seqs > 0 else float(S)\n    eps_hi", "N = float(T)\n    eps_hi"),
    "sequence mean divides by T": ("seq_mean[i] = tot / (b - a)", "seq_mean[i] = tot / e.shape[0]"),
}

PIN_TESTS = [
    lambda: pins.test_entropy_bounds_and_two_forms(),
    lambda: pins.test_against_scipy_log_softmax((5, 3, 7)),
    lambda: pins.test_binary_entropy_closed_form(),
    lambda: [pins.test_brute_force_T3_V4_H2(m, k) for m, k in (("sais", "always"), ("sais", "dynamic"), ("sais", "off"))],
    lambda: [pins.test_clip_quadrants(row) for row in pins.golden("clip")],
    lambda: pins.test_asymmetric_clip_bounds(),
    lambda: pins.test_mask_invariants(),
    lambda: pins.test_threshold_strictness(),
    lambda: pins.test_entropy_scopes_and_sequence_means(),
    lambda: pins.test_mean_nll_special_case(),
    lambda: pins.test_dW_column_sums_vanish_and_dhidden_row_form(),
    lambda: [pins.test_finite_differences(k, "tokens", 0.0) for k in (1.0, 1.0 / 0.85)],
    lambda: pins.test_kl_estimate_closed_forms_and_expectation(),
    lambda: pins.test_kl_term_in_the_decision_stage(),
    lambda: pins.test_finite_differences(1.0, "tokens", 0.3),
    lambda: pins.test_staleness_statistics(),
    lambda: pins.test_group_advantages_closed_forms(),
    lambda: pins.test_sequence_normalisation_closed_forms(),
    lambda: pins.test_finite_differences(1.0, "sequence", 0.0),
]


def load_mutant(old, new):
    text = open(SRC).read()
    assert text.count(old) == 1, f"mutation site not unique: {old!r}"
    mod = types.ModuleType("ulorl_oracle_mutant")
    mod.__file__ = SRC
    sys.modules[mod.__name__] = mod          # dataclasses look their module up by name
    exec(compile(text.replace(old, new), SRC, "exec"), mod.__dict__)
    return mod


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_planted_mistake_is_caught(name, monkeypatch):
    old, new = MUTANTS[name]
    monkeypatch.setattr(pins, "O", load_mutant(old, new))
    caught = 0
    for t in PIN_TESTS:
        try:
            t()
        except (AssertionError, FloatingPointError, ValueError, ZeroDivisionError):
            caught += 1
    assert caught >= 1, f"no pin notices: {name}"


def test_unmutated_oracle_passes_the_same_pins():
    for t in PIN_TESTS:
        t()
