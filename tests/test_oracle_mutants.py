"""Do the oracle's pins notice a mistake?  Plant one in a copy of the oracle and run the pins on it.

Each mutant below is the oracle's source with one plausible slip (a dropped factor, a flipped sign, a
transposed operand, an off-by-one in the ring or in the schedule) compiled into a module of its own.  The
pin tests of tests/test_oracle_pins.py are then run against that module; at least one of them has to fail.
A mutant that survives means the pins leave that part of the oracle unchecked.  Everything here runs on
the CPU and touches only the oracle.
"""
import inspect
import os
import sys
import types

import pytest

from tests import test_oracle_pins as pins

ORACLE_SOURCE = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "oracle", "natural_galore.py")

# (what the slip is, text in the oracle, text of the mutant)
MUTANTS = [
    ("Gram matrix not divided by the number of gradients held",
     "K[i, j] = float(np.sum(history[i] * history[j])) / c", "K[i, j] = float(np.sum(history[i] * history[j]))"),
    ("S built without the 1/lambda", "S = np.eye(c) + K / lam", "S = np.eye(c) + K"),
    ("y = U^T vec(R) without the 1/sqrt(c) of U",
     "y = np.array([float(np.sum(H * R)) / rc for H in history]", "y = np.array([float(np.sum(H * R)) for H in history]"),
    ("U z without the 1/sqrt(c) of U", "Uz += (z[i] / rc) * history[i]", "Uz += z[i] * history[i]"),
    ("sign of the Woodbury correction", "return R / lam - Uz / (lam * lam)", "return R / lam + Uz / (lam * lam)"),
    ("correction scaled by 1/lambda instead of 1/lambda^2", "return R / lam - Uz / (lam * lam)", "return R / lam - Uz / lam"),
    ("leading term not scaled by 1/lambda", "return R / lam - Uz / (lam * lam)", "return R - Uz / (lam * lam)"),
    ("first moment adds the whole gradient", "m = beta1 * m + (1.0 - beta1) * g", "m = beta1 * m + g"),
    ("second moment of g instead of g^2", "v = beta2 * v + (1.0 - beta2) * g * g", "v = beta2 * v + (1.0 - beta2) * g"),
    ("eps outside the square root by default",
     "u = mh / (np.sqrt(vh) + eps) if eps_outside else mh / np.sqrt(vh + eps)",
     "u = mh / np.sqrt(vh + eps) if eps_outside else mh / (np.sqrt(vh) + eps)"),
    ("last singular vectors instead of the first", "return np.ascontiguousarray(U[:, :rp])", "return np.ascontiguousarray(U[:, -rp:])"),
    ("right basis taken from the left singular vectors",
     "return np.ascontiguousarray(Vt[:rp, :].T)", "return np.ascontiguousarray(np.linalg.svd(G.T, full_matrices=False)[2][:rp, :].T)"),
    ("projection without the transpose of P (square P)", "return P.T @ G", "return (P @ G) if P.shape[0] == P.shape[1] else P.T @ G"),
    ("count of gradients held grows past the ring", "self.count = min(self.count + 1, hp.s)", "self.count = self.count + 1"),
    ("ring never wraps onto the oldest slot", "self.head = (self.head + 1) % hp.s", "self.head = min(self.head + 1, hp.s - 1)"),
    ("refresh one step late", "if auto_refresh and hp.T > 0 and self.k % hp.T == 0:", "if auto_refresh and hp.T > 0 and self.k % hp.T == 1 % hp.T:"),
    ("update not scaled by the learning rate", "dW = -hp.lr * back - hp.lr * hp.wd * W", "dW = -back - hp.lr * hp.wd * W"),
    ("update with the wrong sign", "dW = -hp.lr * back - hp.lr * hp.wd * W", "dW = hp.lr * back - hp.lr * hp.wd * W"),
    ("weight decay not scaled by the learning rate", "dW = -hp.lr * back - hp.lr * hp.wd * W", "dW = -hp.lr * back - hp.wd * W"),
    ("weight decay applied to the updated W", "dW = -hp.lr * back - hp.lr * hp.wd * W", "dW = -hp.lr * back - hp.lr * hp.wd * (W - hp.lr * back)"),
    ("Cholesky column without the subtraction of earlier columns",
     "L[i, j] = (S[i, j] - float(np.dot(L[i, :j], L[j, :j]))) / L[j, j]", "L[i, j] = S[i, j] / L[j, j]"),
    ("backward substitution with the untransposed factor",
     "z[i] = (t[i] - float(np.dot(L[i + 1:, i], z[i + 1:]))) / L[i, i]", "z[i] = (t[i] - float(np.dot(L[i, i + 1:], z[i + 1:]))) / L[i, i]"),
    ("bf16 rounding with ties away from zero", "u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000", "u = (u + 0x8000) & 0xFFFF0000"),
    ("bf16 truncation instead of rounding", "u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000", "u = u & 0xFFFF0000"),
    ("square matrices left on the left projection under the short-side rule",
     'self.right = hp.projection == "short_side" and M >= N', 'self.right = hp.projection == "short_side" and M > N'),
    ("right-projected update without the transpose of Q (square Q)",
     "back = u @ self.P.T if self.right else self.P @ u",
     "back = (u @ self.P if self.P.shape[0] == self.P.shape[1] else u @ self.P.T) if self.right else self.P @ u"),
    ("bf16 history rounds the slot about to be overwritten, not the one just used",
     "slot = (self.head - 1) % hp.s", "slot = self.head % hp.s"),
    ("history and moments dropped at every refresh", "reset_history_on_refresh: bool = False", "reset_history_on_refresh: bool = True"),
    ("P kept unrounded", "store_P_as_bf16: bool = True", "store_P_as_bf16: bool = False"),
    ("Philox with nine rounds", "    for _ in range(10):\n        p0 = np.uint64(PHILOX_M0) * c[:, 0]", "    for _ in range(9):\n        p0 = np.uint64(PHILOX_M0) * c[:, 0]"),
    ("Philox round with the two multipliers swapped", "p0 = np.uint64(PHILOX_M0) * c[:, 0]", "p0 = np.uint64(PHILOX_M1) * c[:, 0]"),
    ("rounding bits from the lower halves of the words", "return (words >> np.uint32(16)).reshape(-1)[:n_elements]", "return (words & np.uint32(0xFFFF)).reshape(-1)[:n_elements]"),
    ("second moment rounded to nearest, not stochastically",
     "self.v = stochastic_round_to_bf16(self.v, bits.reshape(self.v.shape))", "self.v = round_to_bf16(self.v)"),
    ("stochastic rounding that always rounds down", "u = (u + bits16.astype(np.uint64).reshape(-1)) & np.uint64(0xFFFF0000)", "u = u & np.uint64(0xFFFF0000)"),
    ("first moment left unrounded under moments_bf16", "            self.m = round_to_bf16(self.m)\n", "            pass\n"),
]


def _pin_cases():
    """Every pin test as (name, function, keyword arguments), parametrised ones expanded."""
    cases = []
    for name, fn in inspect.getmembers(pins, inspect.isfunction):
        if not name.startswith("test_"):
            continue
        marks = [m for m in getattr(fn, "pytestmark", []) if m.name == "parametrize"]
        if not marks:
            cases.append((name, fn, {}))
            continue
        assert len(marks) == 1, name
        names = [n.strip() for n in marks[0].args[0].split(",")]
        for values in marks[0].args[1]:
            values = values if isinstance(values, (tuple, list)) else (values,)
            cases.append((f"{name}{list(values)}", fn, dict(zip(names, values))))
    return cases


def _failing_pins(module):
    failed = []
    saved = pins.orc
    pins.orc = module
    try:
        for name, fn, kwargs in _pin_cases():
            try:
                fn(**kwargs)
            except Exception:      # an assertion, or the mutant breaking outright
                failed.append(name)
    finally:
        pins.orc = saved
    return failed


def _load(source, name):
    mod = types.ModuleType(name)
    mod.__file__ = ORACLE_SOURCE
    sys.modules[name] = mod          # dataclasses looks the module up by name
    try:
        exec(compile(source, ORACLE_SOURCE, "exec"), mod.__dict__)
    finally:
        del sys.modules[name]
    return mod


def test_the_unmodified_copy_passes_every_pin():
    with open(ORACLE_SOURCE) as f:
        source = f.read()
    assert _failing_pins(_load(source, "oracle_copy")) == []


@pytest.mark.filterwarnings("ignore::RuntimeWarning")      # a mutant may take the root of a negative number
@pytest.mark.parametrize("what,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_a_planted_mistake_fails_a_pin(what, old, new):
    with open(ORACLE_SOURCE) as f:
        source = f.read()
    assert source.count(old) == 1, f"mutation site not found exactly once: {old!r}"
    failed = _failing_pins(_load(source.replace(old, new), "oracle_mutant"))
    assert failed, f"no pin notices: {what}"
