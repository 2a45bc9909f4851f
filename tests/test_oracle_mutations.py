"""Plants mistakes in a COPY of the oracle (CPU only) and checks that the pins notice: each
mutated copy is compiled next to the test's temporary files and the pin tests are run against it
in a subprocess, where they must fail. Guards against pins that pass no matter what."""
import os
import shutil
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
ORACLE = os.path.join(ROOT, "oracle")
PINS, NOISE, SGP, NOAVG, F32 = ("tests/test_oracle_pins.py", "tests/test_oracle_noise.py", "tests/test_oracle_sgp.py",
                                 "tests/test_oracle_noaverage.py", "tests/test_oracle_binary32.py")

# (file, text to find, replacement, pin file expected to notice): one plausible slip each
MUTATIONS = [
    ("slowmo_oracle.c", "d = FMA(mu, h[i], g);", "d = FMA(mu, h[i], (real)0) ;", PINS),                      # Nesterov look-ahead term dropped
    ("slowmo_oracle.c", "u = FMA(beta, u, (x0 - xbar) * inv_gam);", "u = FMA(beta, u, (xbar - x0) * inv_gam);", PINS),  # sign of Eq. 2
    ("slowmo_oracle.c", "x0 = FMA(-alpha_gam, u, x0);", "x0 = FMA(-gam, u, x0);", PINS),                      # alpha forgotten in Eq. 3
    ("slowmo_oracle.c", "const real v_hat = v[i] * ibc2;", "const real v_hat = v[i] * ibc1;", PINS),          # wrong bias correction
    ("slowmo_oracle.c", "d = h_hat / (SQRT(v_hat) + eps);", "d = h_hat / SQRT(v_hat + eps);", PINS),          # epsilon inside the root
    ("slowmo_oracle.c", "const real xbar = s / (real)m;", "const real xbar = s / (real)(m + 1);", PINS),      # wrong divisor of the average
    ("slowmo_oracle.c", "const uint32_t from = (i + m - hops % m) % m;", "const uint32_t from = (i + hops) % m;", SGP),  # push direction reversed
    ("slowmo_oracle.c", "u_own[i] = FMA(beta, u_own[i], (x0_own[i] - x[i]) * inv_gam);",
     "u_own[i] = FMA(beta, u_own[i], (x0_own[0] - x[i]) * inv_gam);", NOAVG),                                  # worker index slip
    ("slowmo_noise.c", "case 1: *cos_out = -sin_psi; *sin_out = cos_psi;  break;",
     "case 1: *cos_out = sin_psi; *sin_out = cos_psi;  break;", NOISE),                                        # quadrant sign
    ("slowmo_noise.c", "s ^= s >> 27;", "s ^= s >> 28;", NOISE),                                               # hash shift
    ("slowmo_noise.c", "return z[j & 1];", "return z[0];", NOISE),                                             # sine output never used
    ("slowmo_oracle.c", "pow_b1 = pow_b2 = 1.0;", ";", PINS),                                                   # reset policy keeps the old bias-correction powers
    ("slowmo_oracle.c", "sv = sv + v[i];", "sv = sv + h[i];", PINS),                                            # averaged second moment takes the wrong buffer
    ("slowmo_oracle.c", "const real hbar = sh / (real)m, vbar = sv / (real)m;", "const real hbar = sh, vbar = sv;", PINS),  # buffer sums not divided
    ("slowmo_oracle.c", "h[i] = FMA(b1, h[i], omb1 * g);", "h[i] = FMA(b1, h[i], g);", PINS),                   # (1 - beta_1) forgotten
    ("slowmo_oracle.c", "v[i] = FMA(b2, v[i], omb2 * (g * g));", "v[i] = FMA(b2, v[i], omb2 * g);", PINS),      # gradient not squared
    ("slowmo_oracle.c", "if (cfg->weight_decay != 0.0f) g = FMA((real)cfg->weight_decay, x, g);",
     "if (cfg->weight_decay != 0.0f) g = FMA((real)cfg->weight_decay, g, g);", PINS),                           # L2 term on the gradient instead of x
    ("slowmo_oracle.c", "const double gam_d = (double)(gamma_t ? gamma_t[t] : cfg->gamma);",
     "const double gam_d = (double)cfg->gamma;", PINS),                                                        # learning-rate schedule ignored
    ("slowmo_oracle.c", "for (uint32_t r = m - 1; r > 0; r >>= 1) nq += 1;", "for (uint32_t r = m; r > 0; r >>= 1) nq += 1;", SGP),  # one hop distance too many when m is a power of two
    ("slowmo_noise.c", "float radius = sqrtf(-2.0f * ln_unit24(k1 + 1));", "float radius = sqrtf(-2.0f * ln_unit24(k1 + 2));", NOISE),  # u1 off by one step
    # slips that exist in the binary32 build only (the binary64 pins cannot see them)
    ("slowmo_oracle.c", "#define SQRT(a) sqrtf(a)", "#define SQRT(a) sqrtf(sqrtf(a))", F32),                    # wrong root in the float build
    ("slowmo_oracle.c", "#define FMA(a, b, c) fmaf((a), (b), (c))", "#define FMA(a, b, c) fmaf((a), (b), (float)(int)(c))", F32),  # a cast that truncates
]


def _build_copy(tmp, fname, find, repl):
    for f in ("slowmo_oracle.c", "slowmo_noise.c", "slowmo_oracle.h"):
        shutil.copy(os.path.join(ORACLE, f), tmp)
    path = os.path.join(tmp, fname)
    text = open(path).read()
    assert text.count(find) == 1, f"mutation target not found exactly once: {find}"
    open(path, "w").write(text.replace(find, repl))
    flags = ["-O1", "-std=c11", "-fPIC", "-fopenmp", "-ffp-contract=off", "-D_GNU_SOURCE"]
    objs = []
    for name, src, defs in (("n", "slowmo_noise.c", []), ("a", "slowmo_oracle.c", ["-DORACLE_F64=0"]),
                            ("b", "slowmo_oracle.c", ["-DORACLE_F64=1"])):
        obj = os.path.join(tmp, name + ".o")
        subprocess.check_call(["gcc", *flags, *defs, "-c", os.path.join(tmp, src), "-o", obj])
        objs.append(obj)
    lib = os.path.join(tmp, "libmut.so")
    subprocess.check_call(["gcc", "-shared", "-fopenmp", "-o", lib, *objs, "-lm"])
    return lib


@pytest.mark.parametrize("fname,find,repl,pins", MUTATIONS, ids=[f"{m[0]}:{i}" for i, m in enumerate(MUTATIONS)])
def test_a_planted_mistake_fails_some_pin(tmp_path, fname, find, repl, pins):
    lib = _build_copy(str(tmp_path), fname, find, repl)
    # the second variable tells tests/conftest.py that this run is the mutation harness: a stray
    # SLOWMO_ORACLE_LIB alone is refused there
    env = dict(os.environ, SLOWMO_ORACLE_LIB=lib, SLOWMO_ORACLE_MUTATION_RUN="1")
    run = subprocess.run([sys.executable, "-m", "pytest", pins, "-x", "-q", "-p", "no:cacheprovider",
                          "-k", "not frozen and not mutation and not every_radius"], cwd=ROOT, env=env,
                         capture_output=True, timeout=600)
    assert run.returncode == 1, "the pins did not notice: " + run.stdout.decode()[-1500:]
