"""Plants one plausible mistake at a time in a COPY of the CPU oracle (a dropped factor, a wrong sign, a squared
distance, a transposed index ...) and checks that the pin battery notices each of them.  Nothing here touches a GPU."""
import importlib.util
import os
import shutil

import pytest

from pin_battery import run_battery

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
ORACLE = os.path.join(ROOT, "oracle")

MUTATIONS = [
    ("squared distance in the softmax", "    D[j] = g_squared ? s : sqrt(s);", "    D[j] = s;"),
    ("temperature dropped from the softmax", "A[j] = exp(-(D[j] - dmin) / tau);", "A[j] = exp(-(D[j] - dmin));"),
    ("M-step not normalised by the column sum", "C_plus[j * d + a] = N[j * d + a] / S[j];",
     "C_plus[j * d + a] = N[j * d + a] / (double)m;"),
    ("1/tau dropped from the codebook gradient", "pg[j * d + a] += A[j] * Gi[a] + (e / tau) * n[a];",
     "pg[j * d + a] += A[j] * Gi[a] + e * n[a];"),
    ("direct term dropped from the codebook gradient", "pg[j * d + a] += A[j] * Gi[a] + (e / tau) * n[a];",
     "pg[j * d + a] += (e / tau) * n[a];"),
    ("sign of the softmax term in dL/dW", "dW[i * d + a] += A[j] * u[j * d + a] * inv_s - (e / tau) * n[a];",
     "dW[i * d + a] += A[j] * u[j * d + a] * inv_s + (e / tau) * n[a];"),
    ("A u / S term dropped from dL/dW", "dW[i * d + a] += A[j] * u[j * d + a] * inv_s - (e / tau) * n[a];",
     "dW[i * d + a] += - (e / tau) * n[a];"),
    ("p not divided by the column sum", "  return s / S[j];", "  return s;"),
    ("p uses the centroid instead of F", "s += u[j * d + a] * (w[a] - F[j * d + a]);", "s += u[j * d + a] * w[a];"),
    ("mean subtraction dropped in the adjoint", "double e = A[j] * (p[j] - s);", "double e = A[j] * p[j];"),
    ("unit vector points the wrong way", "n[a] = (Dj > 0.0) ? (w[a] - cj[a]) / Dj : 0.0;",
     "n[a] = (Dj > 0.0) ? (cj[a] - w[a]) / Dj : 0.0;"),
    ("averaging weight applied to the wrong term", "un[t] = alpha * (Ju[t] + g[t]) + (1.0 - alpha) * u[t];",
     "un[t] = (1.0 - alpha) * (Ju[t] + g[t]) + alpha * u[t];"),
    ("Wq uses transposed attention index", "for (int j = 0; j < k; ++j) s += A[j] * C[j * d + a];",
     "for (int j = 0; j < k; ++j) s += A[k - 1 - j] * C[j * d + a];"),
]

# the same for the squared-distance variant (the battery then runs with the variant switched on)
MUTATIONS_SQUARED = [
    ("variant ignores the switch in the distance", "    D[j] = g_squared ? s : sqrt(s);", "    D[j] = sqrt(s);"),
    ("factor 2 of the squared distance's gradient dropped", "n[a] = 2.0 * (w[a] - cj[a]);", "n[a] = (w[a] - cj[a]);"),
    ("squared distance's gradient normalised like the unit vector", "n[a] = 2.0 * (w[a] - cj[a]);",
     "n[a] = (Dj > 0.0) ? (w[a] - cj[a]) / sqrt(Dj) : 0.0;"),
    ("sign of the squared distance's gradient", "n[a] = 2.0 * (w[a] - cj[a]);", "n[a] = 2.0 * (cj[a] - w[a]);"),
    ("mean subtraction dropped in the adjoint", "double e = A[j] * (p[j] - s);", "double e = A[j] * p[j];"),
    ("1/tau dropped from the codebook gradient", "pg[j * d + a] += A[j] * Gi[a] + (e / tau) * n[a];",
     "pg[j * d + a] += A[j] * Gi[a] + e * n[a];"),
]


def _load_mutant(tmp_path, old, new):
    src = open(os.path.join(ORACLE, "idkm_ref.c")).read()
    assert src.count(old) == 1, f"mutation target not unique: {old!r} x{src.count(old)}"
    d = tmp_path / "mutant"
    d.mkdir()
    (d / "idkm_ref.c").write_text(src.replace(old, new))
    shutil.copy(os.path.join(ORACLE, "idkm_ref.py"), d / "idkm_ref.py")
    spec = importlib.util.spec_from_file_location("idkm_ref_mutant", str(d / "idkm_ref.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


def test_unmutated_oracle_passes_the_battery():
    from oracle import idkm_ref as R
    assert run_battery(R) == []
    assert run_battery(R, squared=True) == []
    assert R.get_squared() is False          # the battery leaves the oracle in the published setting


@pytest.mark.parametrize("name,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_battery_catches_planted_mistake(tmp_path, name, old, new):
    mutant = _load_mutant(tmp_path, old, new)
    failed = run_battery(mutant)
    assert failed, f"no pin noticed: {name}"


@pytest.mark.parametrize("name,old,new", MUTATIONS_SQUARED, ids=[m[0] for m in MUTATIONS_SQUARED])
def test_battery_catches_planted_mistake_in_the_squared_variant(tmp_path, name, old, new):
    mutant = _load_mutant(tmp_path, old, new)
    failed = run_battery(mutant, squared=True)
    assert failed, f"no pin noticed: {name}"
