"""Mutation check of the oracle's pins: a plausible mistake in the oracle must fail a pin.

Each entry rewrites one line of the oracle's source (a tie rule, a denominator, a sign, an order),
loads the result as a throw-away module and runs the pin tests against it.  A mutation that no pin
notices means the pins do not fix that line.  The oracle on disk is never modified.
"""
import inspect
import os
import types

import pytest

from oracle import eb_oracle as O
from tests import test_oracle_pins as P

SRC = inspect.getsource(O)

# (name, text in the oracle, replacement)
MUTATIONS = [
    # the top-up of the O(n) policies to m members (Section 4.2: |RunSet| >= m)
    ("top-up takes the lowest-U member", "if best_u is None or _u_greater(u, best_u):",
     "if best_u is None or _u_greater(best_u, u):"),
    ("top-up ties go to the highest index", "if best_u is None or _u_greater(u, best_u):",
     "if best_u is None or not _u_greater(best_u, u):"),
    ("top-up adds the whole pool", "chosen |= 1 << best_j", "chosen |= pool"),
    ("top-up adds the lowest index", "            if best_u is None or _u_greater(u, best_u):\n",
     "            if best_u is None:\n"),
    ("no work counts as U = 0", "an, ad = a if a[1] != 0 else (1, 1)\n    bn, bd = b if b[1] != 0 else (1, 1)",
     "an, ad = a if a[1] != 0 else (0, 1)\n    bn, bd = b if b[1] != 0 else (0, 1)"),
    # routing
    ("top-k ties to the higher index", 'order = np.argsort(-logits, axis=1, kind="stable")',
     'order = np.argsort(-logits[:, ::-1], axis=1, kind="stable"); order = logits.shape[1] - 1 - order'),
    ("renormalisation flag inverted", "    if renorm_topk:\n        w = p / p.sum(axis=1, keepdims=True)",
     "    if not renorm_topk:\n        w = p / p.sum(axis=1, keepdims=True)"),
    ("loads count tokens, not assignments", "np.add.at(mb_load[j], dev[sel], 1)",
     "np.add.at(mb_load[j], dev[idx[tok_off[j]:tok_off[j + 1], 0]], 1)"),
    # utilisation and MaxUtil
    ("utilisation without D", "return sum(w), len(w) * effective_workload(w)", "return sum(w), effective_workload(w)"),
    ("MaxUtil ties to the larger mask", 'return (u, bin(cands[i]).count("1"), -cands[i])',
     'return (u, bin(cands[i]).count("1"), cands[i])'),
    ("MaxUtil ties to the smaller set", 'return (u, bin(cands[i]).count("1"), -cands[i])',
     'return (u, -bin(cands[i]).count("1"), -cands[i])'),
    ("MaxUtil needs more than m", 'if bin(mask).count("1") >= m:', 'if bin(mask).count("1") > m:'),
    # CumUtil / DiffPeak
    ("CumUtil accepts an equal U",
     "if _u_greater(utilisation(_joint(mb_load, run | (1 << j))), utilisation(_joint(mb_load, run))):",
     "if not _u_greater(utilisation(_joint(mb_load, run)), utilisation(_joint(mb_load, run | (1 << j)))):"),
    ("peak device ties to the higher index", "        if w[d] > w[best]:", "        if w[d] >= w[best]:"),
    # grouping
    ("layer-major group table",
     "    for d in range(D):\n        for l in active:\n            for e in range(E):",
     "    for l in active:\n      for d in range(D):\n        if True:\n            for e in range(E):"),
    ("home device rounds up", "return (t_local * D) // T_j", "return min(D - 1, -(-(t_local * D) // T_j))"),
    ("rows of a group in reverse token order",
     "        for t in range(tok_off[j], tok_off[j + 1]):\n            for k in range(K):",
     "        for t in reversed(range(tok_off[j], tok_off[j + 1])):\n            for k in range(K):"),
    # expert MLP and aggregation
    ("gate and up swapped", "a = silu(g) * u", "a = silu(u) * g"),
    ("SiLU sign", "return g / (1.0 + np.exp(-g))", "return g / (1.0 + np.exp(g))"),
    ("gate weights not applied", "acc = acc + dtype(topk_w[t, k]) * y[pos[t, k]].astype(dtype)",
     "acc = acc + y[pos[t, k]].astype(dtype)"),
    ("shared experts dropped from the sum",
     "        for s in range(S):\n            acc = acc + y[pos[t, K + s]].astype(dtype)",
     "        for s in range(0):\n            acc = acc + y[pos[t, K + s]].astype(dtype)"),
    ("residual missing", "out[t] = acc + residual[t].astype(dtype)", "out[t] = acc"),
    ("residual subtracted", "out[t] = acc + residual[t].astype(dtype)", "out[t] = acc - residual[t].astype(dtype)"),
    # Algorithm 1 and the metrics
    ("finished micro-batches stay in the pool", "            if l[j] >= L:\n                pool &= ~(1 << j)",
     "            if l[j] > L:\n                pool &= ~(1 << j)"),
    ("each-alone capacity uses the joint load",
     'cap = D * sum(effective_workload(w) for s in steps for w in s["member_loads"].values())',
     'cap = D * sum(effective_workload(s["joint_load"]) for s in steps)'),
    ("same-peak count compares with the first layer", "if all(peaks[l + i] == peaks[l] for i in range(1, n)):",
     "if all(peaks[l + i] == peaks[0] for i in range(1, n)):"),
]


def _pin_calls():
    """Every pin test as a list of (label, zero-argument callable), parametrised ones expanded."""
    calls = []
    for name, fn in sorted(vars(P).items()):
        if not name.startswith("test_") or not callable(fn):
            continue
        marks = [mk for mk in getattr(fn, "pytestmark", []) if mk.name == "parametrize"]
        if not marks:
            calls.append((name, fn))
            continue
        assert len(marks) == 1
        for value in marks[0].args[1]:
            calls.append((f"{name}[{value.get('name', '?') if isinstance(value, dict) else value}]",
                          lambda fn=fn, value=value: fn(value)))
    return calls


def _first_failing_pin(module):
    saved = P.O
    P.O = module
    try:
        for label, call in _pin_calls():
            try:
                call()
            except Exception:                                  # noqa: BLE001 - any failure is a catch
                return label
        return None
    finally:
        P.O = saved


def test_unmutated_oracle_passes_through_this_runner():
    assert _first_failing_pin(O) is None


@pytest.mark.parametrize("name,old,new", MUTATIONS, ids=[mu[0] for mu in MUTATIONS])
def test_mutation_is_caught(name, old, new):
    assert SRC.count(old) >= 1, f"pattern of mutation '{name}' is no longer in the oracle"
    mod = types.ModuleType("eb_oracle_mutant")
    mod.__file__ = os.path.join(os.path.dirname(O.__file__), "eb_oracle_mutant.py")
    exec(compile(SRC.replace(old, new, 1), mod.__file__, "exec"), mod.__dict__)
    caught_by = _first_failing_pin(mod)
    assert caught_by is not None, f"no pin notices: {name}"
