"""The pins must notice a plausible mistake anywhere in the oracle.

Each case plants one mistake in a temporary copy of the oracle's C source (on
the CPU, never in the CUDA code), rebuilds it and expects the pin tests to fail.
"""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "adascale_oracle.c")

MUTATIONS = [
    ("divide by S instead of S-1", "double sigma2 = D / (double)(S - 1);", "double sigma2 = D / (double)S;"),
    ("sign of the mu^2 correction", "N - sigma2 / (double)S;", "N + sigma2 / (double)S;"),
    ("non-strict step boundary", "if (t > lr->w[i])", "if (t >= lr->w[i])"),
    ("lr read at tau, not floor(tau)", ": floor(st->tau);", ": st->tau;"),
    ("weight decay dropped", "(gbar[j] + lambda * w[j])", "(gbar[j])"),
    ("ascent instead of descent", "w[j] - eta * vj", "w[j] + eta * vj"),
    ("momentum factor dropped", "rho * v[j] +", "v[j] +"),
    ("average weights swapped", "th * prev + (1.0 - th) * sample", "th * sample + (1.0 - th) * prev"),
    ("gain denominator transposed", "s / (double)S + m", "s + m / (double)S"),
    ("theta rule constant", "(double)cfg->S / 1000.0", "(double)cfg->S / 100.0"),
    ("clock adds 1, not r", "st->tau + r;", "st->tau + 1.0;"),
    ("bf16 shift", "[j] << 16;", "[j] << 15;"),
    ("norm of mean not squared", "nn += mean * mean;", "nn += mean;"),
    ("variance clamp missing", "if (sigma2 < cfg->eps)", "if (0)"),
    ("mean clamp missing", "if (mu2 < 0.0)", "if (0)"),
    ("eta without the gain", "st->eta = r * st->lr;", "st->eta = st->lr;"),
    ("mean divides by S-1", "double mean = sum / (double)S;", "double mean = sum / (double)(S - 1);"),
    ("warm start missing", "if (theta < th)", "if (1)"),
    ("exponent not scaled by T_S1", "pow(lr->d, t / lr->T_S1)", "pow(lr->d, t)"),
    ("lagged r_0", ": 1.0;\n        st->n += 1;\n        st->avg_a = moving_average(st->avg_a, sigma2",
     ": 2.0;\n        st->n += 1;\n        st->avg_a = moving_average(st->avg_a, sigma2"),
    ("ratio-mode r_0", "(st->avg_a + cfg->eps) / (st->avg_b + cfg->eps) : 1.0;",
     "(st->avg_a + cfg->eps) / (st->avg_b + cfg->eps) : 2.0;"),
    ("ratio-mode lagged gain taken after the update", "? r_prior\n                                              : (st->avg_a + cfg->eps)",
     "? (st->avg_a + cfg->eps) / (st->avg_b + cfg->eps)\n                                              : (st->avg_a + cfg->eps)"),
    ("ratio-mode eps missing from the lagged gain", "double r_prior = st->n > 0 ? (st->avg_a + cfg->eps) / (st->avg_b + cfg->eps)",
     "double r_prior = st->n > 0 ? (st->avg_a) / (st->avg_b)"),
]


@pytest.mark.parametrize("name,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_pins_catch(tmp_path, name, old, new):
    src = open(SRC).read()
    assert src.count(old) == 1, "mutation target must be unique: %r" % old
    bad = tmp_path / "mutant.c"
    bad.write_text(src.replace(old, new))
    env = dict(os.environ, ADASCALE_ORACLE_SRC=str(bad))
    res = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_oracle_pins.py"),
                          "-x", "-q", "-k", "not unbiased", "-p", "no:cacheprovider"],
                         cwd=ROOT, env=env, capture_output=True, text=True)
    assert res.returncode == 1, "pins did not notice: %s\n%s" % (name, res.stdout[-2000:])
