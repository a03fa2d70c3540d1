"""Do the pins bite?  Each case plants one plausible mistake in a COPY of the oracle's C source
(a wrong comparison, a dropped term, a wrong sign, a transposed mask, an off-by-one), builds it, and
runs the pin tests against that library in a child process: they must fail.  The mistakes live
only in the temporary copy; nothing here touches the GPU."""
import os
import subprocess
import sys
import tempfile
from concurrent.futures import ThreadPoolExecutor

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "jacobi_oracle.c")

# (name, text in the oracle, planted replacement)
MUTANTS = [
    ("hidden mask strict", ": (m->deg[l + 1][i] >= m->deg[l][j]);", ": (m->deg[l + 1][i] > m->deg[l][j]);"),
    ("output mask not strict", "(l == L) ? (m->deg[l + 1][i] > m->deg[l][j])", "(l == L) ? (m->deg[l + 1][i] >= m->deg[l][j])"),
    ("mask transposed", ": (m->deg[l + 1][i] >= m->deg[l][j]);", ": (m->deg[l + 1][i] <= m->deg[l][j]);"),
    ("bias dropped", "return acc + (double)m->b[l][i];", "return acc;"),
    ("inverse CDF reversed", "return noise[0] < p ? 1 : 0;", "return noise[0] > p ? 1 : 0;"),
    ("logistic threshold reversed", "return s > 0.0f ? 1 : 0;", "return s < 0.0f ? 1 : 0;"),
    ("noise subtracted in argmax", "float v = nz[c] + noise[c];\n        if (v > best_v)", "float v = nz[c] - noise[c];\n        if (v > best_v)"),
    ("bf16 truncation instead of nearest-even", "bits += 0x7fffu + lsb;", "bits += 0u * lsb;"),
    ("GS-Jacobi updates beyond its block", "memcpy(x + a, next + a, (size_t)len);", "memcpy(x + a, next + a, (size_t)(T - a));"),
    ("Jacobi-GS reads the new iterate before the block", "            memcpy(y, prev, (size_t)T);\n            sweep(m, y, a, b, noise, nk);", "            memcpy(y, x, (size_t)T);\n            sweep(m, y, a, b, noise, nk);"),
    ("conv centre tap type A everywhere", "keep = l == 0 ? (gi < go) : (gi <= go);", "keep = (gi < go);"),
    ("conv keeps the tap to the right", "else if (ky == 1 && kx == 0) keep = 1;", "else if (ky == 1 && kx != 1) keep = 1;"),
    ("Jacobi cap one short", "int cap = (max_iters > 0 && max_iters < T) ? max_iters : T;", "int cap = (max_iters > 0 && max_iters < T) ? max_iters : T - 1;"),
    ("sweep starts units one degree late", "if (m->deg[l + 1][i] == t)", "if (m->deg[l + 1][i] == t - 1)"),
    ("Gumbel margin always zero", "    return top - second;", "    return 0.0f;"),
    ("runner-up not kept when the top moves", "if (v > top) { second = top; top = v; }", "if (v > top) { top = v; }"),
    ("logistic margin with the wrong sign", "return fabsf(nz[0] + noise[0]);", "return fabsf(nz[0] - noise[0]);"),
    ("inverse-CDF margin measured to the far boundary", "cum[x] / tot - u < gap) gap", "cum[x] / tot - u > gap) gap"),
    ("categorical inverse CDF not strict", "if (target < cum[c]) return c;", "if (target <= cum[c]) return c;"),
    ("cumulative sum starts one class late", "for (int c = 0; c < C; ++c) { run += exp((double)nz[c] - mx); cum[c] = run; }",
     "for (int c = 0; c < C; ++c) { cum[c] = run; run += exp((double)nz[c] - mx); }"),
    ("softmax without the logits' scale", "run += exp((double)nz[c] - mx); cum[c] = run; }", "run += exp(0.5 * ((double)nz[c] - mx)); cum[c] = run; }"),
    ("custom degrees ignored", "? hidden_deg[l - 1][j]", "? 1 + (int)(((long long)j * (T - 1)) / m->n[l])"),
    ("continuous state: log-scale used as the scale", "(double)zt[0] + exp((double)zt[1]) * (double)eps_t", "(double)zt[0] + (double)zt[1] * (double)eps_t"),
    ("continuous state: noise subtracted", "(double)zt[0] + exp((double)zt[1]) * (double)eps_t", "(double)zt[0] - exp((double)zt[1]) * (double)eps_t"),
    ("continuous state: mean change instead of the largest", "            if (!(d <= dmax)) dmax = d;                 /* a NaN difference counts as a change */", "            dmax += d / (float)T;"),
    ("continuous state: bf16 model reads unrounded inputs", "ws.a[0][d] = m->prec == ORC_PREC_BF16 ? round_bf16(x[d]) : x[d];", "ws.a[0][d] = x[d];"),
    ("continuous state: GS-Jacobi looks at the whole iterate", "            for (int t = a; t < b; ++t) {\n                float d = fabsf(next[t] - x[t]);", "            for (int t = 0; t < T; ++t) {\n                float d = fabsf(next[t] - x[t]);"),
]


def _run_mutant(case):
    name, old, new = case
    text = open(SRC).read()
    assert text.count(old) >= 1, f"mutant '{name}': the oracle no longer contains the text to replace"
    with tempfile.TemporaryDirectory() as d:
        c_path, so_path = os.path.join(d, "mutant.c"), os.path.join(d, "mutant.so")
        open(c_path, "w").write(text.replace(old, new, 1))
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-shared", "-fPIC", "-o", so_path, c_path, "-lm"])
        env = dict(os.environ, ORACLE_LIB=so_path)
        r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                            os.path.join(ROOT, "tests", "test_oracle_pins.py"),
                            os.path.join(ROOT, "tests", "test_oracle_solvers.py"),
                            os.path.join(ROOT, "tests", "test_oracle_real.py")],
                           env=env, cwd=ROOT, capture_output=True, text=True, timeout=600)
    return name, r.returncode, r.stdout[-300:]


def test_every_planted_mistake_fails_a_pin():
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        results = list(ex.map(_run_mutant, MUTANTS))
    survivors = [name for name, rc, _ in results if rc == 0]
    assert not survivors, f"these mistakes pass every pin: {survivors}"


def test_the_unmodified_oracle_passes_under_the_same_harness():
    name, rc, tail = _run_mutant(("none", "/*", "/*"))
    assert rc == 0, tail
