"""The pins must be sharp: a plausible mistake planted in the oracle's arithmetic has to fail
at least one of them.  Each case copies oracle/ to a scratch directory, applies one textual
mutation to dsa3d_oracle.c (a wrong sign, a swapped factor, a shifted window, an off-by-one
at the grid edge, a dropped scale ...), and runs the pin suite against the copy in a
subprocess; the suite must report a failure."""
import os
import shutil
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

MUTATIONS = [
    ("sign of the weight derivative", "double prod = cc[a] ? 1.0 : -1.0;", "double prod = cc[a] ? -1.0 : 1.0;"),
    ("dV uses dS instead of alpha", "cf[1] = alpha[p];", "cf[1] = dS[p];"),
    ("window centred one cell off", "b[0] = u - window[0] / 2;", "b[0] = u - (window[0] - 1) / 2;"),
    ("position -1 treated as dead", "if (!(pi >= -1.0f) || !(pi < (float)size[a]))", "if (!(pi > -1.0f) || !(pi < (float)size[a]))"),
    ("last grid index treated as outside", "if (idx[a] < 0 || idx[a] > size[a] - 1) ok = 0;", "if (idx[a] < 0 || idx[a] >= size[a] - 1) ok = 0;"),
    ("logit not scaled by 1/sqrt(d)", "s[p] = dot * scale;", "s[p] = dot;"),
    ("weights swapped between near and far corner", "g->wt[a][0] = 1.0 - f;\n        g->wt[a][1] = f;", "g->wt[a][0] = f;\n        g->wt[a][1] = 1.0 - f;"),
    ("dead samples dropped from the softmax", "for (int p = 0; p < P; ++p) l += exp(s[p] - mx);", "for (int p = 0; p < P; ++p) if (s[p] != 0.0) l += exp(s[p] - mx);"),
    ("delta term missing from dS", "dS[p] = alpha[p] * (g[p] - delta);", "dS[p] = alpha[p] * g[p];"),
    ("dK scatter misses the scale", "cf[0] = scale * dS[p];", "cf[0] = dS[p];"),
    ("window cells enumerated y-minor instead of x-minor", "int w = p % window[2];\n    int v = (p / window[2]) % window[1];", "int v = p % window[1];\n    int w = (p / window[1]) % window[2];"),
]


@pytest.mark.parametrize("label,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_a_planted_mistake_fails_a_pin(label, old, new, tmp_path):
    work = tmp_path / "mut"
    (work / "tests").mkdir(parents=True)
    shutil.copytree(os.path.join(ROOT, "oracle"), work / "oracle",
                    ignore=shutil.ignore_patterns("*.so", "__pycache__"))
    shutil.copytree(os.path.join(ROOT, "paper_2607_22696_b200"), work / "paper_2607_22696_b200",
                    ignore=shutil.ignore_patterns("*.so", "__pycache__", "csrc"))
    for name in ("test_oracle_pins.py", "conftest.py"):
        shutil.copy(os.path.join(ROOT, "tests", name), work / "tests" / name)
    src = work / "oracle" / "dsa3d_oracle.c"
    text = src.read_text()
    assert text.count(old) >= 1, f"mutation target not found: {old!r}"
    src.write_text(text.replace(old, new))
    res = subprocess.run([sys.executable, "-m", "pytest", "tests/test_oracle_pins.py", "-x", "-q",
                          "-p", "no:cacheprovider"], cwd=work, capture_output=True, text=True, timeout=600)
    assert res.returncode != 0, f"no pin noticed: {label}\n{res.stdout[-400:]}"
    assert "failed" in res.stdout
