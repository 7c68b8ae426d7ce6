"""Mutation check of the oracle's pins: each entry plants one plausible mistake
in a copy of ``oracle/psops_ref.c`` (on the CPU, never in the CUDA path),
builds it, and requires that the pin suite fails against that build."""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

import pytest

from conftest import ROOT

SRC = os.path.join(ROOT, "oracle", "psops_ref.c")
CFLAGS = ["-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-fPIC", "-shared"]

# multi-line passages of the oracle that several mutants rewrite
_QUAD_L2R = ("double a = quad_term(x, dvec, tvec, j, N);\n"
             "            a = a + quad_term(x, dvec, tvec, j + 1, N);\n"
             "            a = a + quad_term(x, dvec, tvec, j + 2, N);\n"
             "            a = a + quad_term(x, dvec, tvec, j + 3, N);")
_GROUPS_IN_ORDER = ("for (int grp = 0; grp < 32; ++grp) {\n"
                    "        double a[32];\n"
                    "        for (int l = 0; l < 32; ++l) a[l] = slot[grp * 32 + l];\n"
                    "        double gsum = butterfly32(a);\n"
                    "        total = (grp == 0) ? gsum : total + gsum;")

MUTANTS = [
    ("philox multiplier", "0xD2511F53u", "0xD2511F52u"),
    ("philox key increment", "0xBB67AE85u", "0xBB67AE86u"),
    ("philox nine rounds", "round < 10", "round < 9"),
    ("philox key bumped before the first round", "if (round > 0) {", "if (round >= 0) {"),
    ("philox hi halves not crossed", "uint32_t n0 = hi_b ^ c1 ^ k0;", "uint32_t n0 = hi_a ^ c1 ^ k0;"),
    ("uniform takes 23 bits", "(float)(word >> 8) * 0x1p-24f", "(float)(word >> 9) * 0x1p-23f"),
    ("counter uses d, not d >> 1", "(uint32_t)(d >> 1), i, s, 0u", "(uint32_t)d, i, s, 0u"),
    ("counter words i and s swapped", "(uint32_t)(d >> 1), i, s, 0u", "(uint32_t)(d >> 1), s, i, 0u"),
    ("odd/even lanes swapped", "if (d & 1u) {", "if (!(d & 1u)) {"),
    ("r1 and r2 swapped", "*r1 = psops_ref_uniform(o[0]);\n        *r2 = psops_ref_uniform(o[1]);",
     "*r2 = psops_ref_uniform(o[0]);\n        *r1 = psops_ref_uniform(o[1]);"),
    ("seed halves swapped", "(uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32)",
     "(uint32_t)(seed >> 32), (uint32_t)(seed & 0xffffffffu)"),
    ("argmin takes the last minimum", "if (loss[i] < loss[g] ||", "if (loss[i] <= loss[g] ||"),
    ("argmin lets NaN stay", "|| (incumbent_nan && !candidate_nan)) g = i;", ") g = i;"),
    ("equal loss improves pBest", "(uint8_t)(loss[i] < pbest_loss[i])", "(uint8_t)(loss[i] <= pbest_loss[i])"),
    ("pBest_loss not updated", "if (improved[i]) pbest_loss[i] = loss[i];", ""),
    ("local term sign", "float dl = pp - xo;", "float dl = xo - pp;"),
    ("global term sign", "float dg = gb - xo;", "float dg = xo - gb;"),
    ("search terms cross-paired", "fmaf(t2, dg, fmaf(t1, dl, a0))", "fmaf(t1, dg, fmaf(t2, dl, a0))"),
    ("inner fma unfused", "fmaf(t2, dg, fmaf(t1, dl, a0))", "fmaf(t2, dg, t1 * dl + a0)"),
    ("inertia dropped", "float a0 = m * vo;", "float a0 = vo;"),
    ("position subtracts", "*xn = xo + vnew;", "*xn = xo - vnew;"),
    ("lambda multiplies", "const float k1 = c1 / lambda;", "const float k1 = c1 * lambda;"),
    ("lambda missing on the global term", "const float k2 = c2 / lambda;", "const float k2 = c2;"),
    ("pBest used before its update", "const float pp = improved[i] ? xo : p[at];", "const float pp = p[at];"),
    ("pBest receives the new weight", "if (improved[i]) p[at] = xo;", "if (improved[i]) p[at] = xn;"),
    ("gBest read from the live row", "r1, r2, xo, vo, pp, gb[j],",
     "r1, r2, xo, vo, pp, x[(size_t)g * (size_t)ld + (size_t)j],"),
    ("gBest is the arg-max", "const int g = psops_ref_argmin(loss, K);",
     "int g = 0; for (int q = 1; q < K; ++q) if (loss[q] > loss[g]) g = q;"),
    ("step counter ignored", "psops_ref_draw(seed, s, (uint32_t)i, d, &r1, &r2)",
     "psops_ref_draw(seed, 0u, (uint32_t)i, d, &r1, &r2)"),
    ("element index map ignored", "elem_index ? (uint64_t)elem_index[j] : (uint64_t)j", "(uint64_t)j"),
    ("schedule sign", "(double)m_max\n             - (double)t", "(double)m_max\n             + (double)t"),
    ("schedule not clamped", "if (t > t_max) t = t_max;", ""),
    ("average divides by K-1", "acc / (float)K", "acc / (float)(K > 1 ? K - 1 : 1)"),
    ("average counts row 0 twice", "for (int k = 1; k < K; ++k)\n            acc = acc + x[",
     "for (int k = 0; k < K; ++k)\n            acc = acc + x["),
    ("ssgd counts worker 0 twice", "for (int k = 1; k < K; ++k)\n            acc = acc + grad[",
     "for (int k = 0; k < K; ++k)\n            acc = acc + grad["),
    ("history: equal loss replaces the remembered best", "if (!*hist_valid || loss[g] < *hist_loss) {",
     "if (!*hist_valid || loss[g] <= *hist_loss) {"),
    ("history: empty memory not filled", "if (!*hist_valid || loss[g] < *hist_loss) {",
     "if (loss[g] < *hist_loss) {"),
    ("history: remembered row not used", "memcpy(gb, hist_row, sizeof(float) * (size_t)n);     /* keep", "/* keep"),
    ("history: remembers the post-update row", "memcpy(hist_row, gb, sizeof(float) * (size_t)n);     /* new best in history */",
     "/* new best in history */"),
    ("ssgd not divided by the worker count", "const float scale = alpha / (float)K;", "const float scale = alpha;"),
    ("ssgd subtracts", "const float wn = w[j] + step;", "const float wn = w[j] - step;"),
    ("ssgd ignores the gradient stride", "acc = acc + grad[(size_t)k * (size_t)grad_ld + (size_t)j];",
     "acc = acc + grad[(size_t)k * (size_t)ld + (size_t)j];"),
    ("fitness error not squared", "float e2 = e * e;", "float e2 = e;"),
    ("fitness uses tvec as weight", "float term = dvec[j] * e2;", "float term = tvec[j] * e2;"),
    ("fitness drops the last element of a quad", "a = a + quad_term(x, dvec, tvec, j + 3, N);", ""),
    ("fitness drops tiles beyond the slots", "slot[mt % 1024] = slot[mt % 1024] + butterfly32(q);",
     "if (mt < 1024) slot[mt] = slot[mt] + butterfly32(q);"),
    # summation order and term rounding of the fitness (the hand-worked cancellation cases)
    ("fitness butterfly stages 1 -> 16", "for (int off = 16; off >= 1; off >>= 1) {",
     "for (int off = 1; off <= 16; off <<= 1) {"),
    ("fitness quad added right to left", _QUAD_L2R,
     "double a = quad_term(x, dvec, tvec, j + 3, N);\n"
     "            a = a + quad_term(x, dvec, tvec, j + 2, N);\n"
     "            a = a + quad_term(x, dvec, tvec, j + 1, N);\n"
     "            a = a + quad_term(x, dvec, tvec, j, N);"),
    ("fitness quad added pairwise", _QUAD_L2R,
     "double a = (quad_term(x, dvec, tvec, j, N) + quad_term(x, dvec, tvec, j + 1, N))\n"
     "                   + (quad_term(x, dvec, tvec, j + 2, N) + quad_term(x, dvec, tvec, j + 3, N));"),
    ("fitness quad accumulated in fp32", "double a = quad_term(x, dvec, tvec, j, N);",
     "float a = (float)quad_term(x, dvec, tvec, j, N);"),
    ("fitness tile quads added one after another", "slot[mt % 1024] = slot[mt % 1024] + butterfly32(q);",
     "{ double ts = q[0]; for (int l = 1; l < 32; ++l) ts = ts + q[l]; slot[mt % 1024] = slot[mt % 1024] + ts; }"),
    ("fitness 512 slots", "slot[mt % 1024] = slot[mt % 1024] + butterfly32(q);",
     "slot[mt % 512] = slot[mt % 512] + butterfly32(q);"),
    ("fitness tiles visited in decreasing order", "for (int64_t mt = 0; mt < tiles; ++mt) {",
     "for (int64_t mt = tiles - 1; mt >= 0; --mt) {"),
    ("fitness slots of a group added one after another", "double gsum = butterfly32(a);",
     "double gsum = a[0]; for (int l = 1; l < 32; ++l) gsum = gsum + a[l];"),
    ("fitness group sums added in reverse", _GROUPS_IN_ORDER,
     _GROUPS_IN_ORDER.replace("int grp = 0; grp < 32; ++grp", "int grp = 31; grp >= 0; --grp")
                     .replace("(grp == 0) ?", "(grp == 31) ?")),
    ("fitness group sums combined by a butterfly", "total = (grp == 0) ? gsum : total + gsum;",
     "slot[grp] = gsum; if (grp == 31) total = butterfly32(slot);"),
    ("fitness term evaluated as (d*e)*e", "float e2 = e * e;\n    float term = dvec[j] * e2;",
     "float term = (dvec[j] * e) * e;"),
    ("fitness term evaluated in fp64", "return (double)term;",
     "(void)term; { double ed = (double)x[j] - (double)tvec[j]; return (double)(float)((double)dvec[j] * (ed * ed)); }"),
    ("fitness square kept in fp64", "float term = dvec[j] * e2;",
     "(void)e2; float term = (float)((double)dvec[j] * ((double)e * (double)e));"),
]


def _run_pins(lib_path):
    env = dict(os.environ, PSOPS_REF_LIB=lib_path, OMP_NUM_THREADS="2")
    return subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_oracle_pins.py"),
                           "-x", "-q", "-p", "no:cacheprovider"], env=env, cwd=ROOT,
                          capture_output=True, text=True, timeout=600)


def _mutant_survives(args):
    name, old, new, tmp = args
    text = open(SRC).read()
    assert text.count(old) == 1, f"mutation '{name}': pattern must occur exactly once"
    path_c = os.path.join(tmp, f"m_{abs(hash(name))}.c")
    path_so = path_c[:-2] + ".so"
    with open(path_c, "w") as fh:
        fh.write(text.replace(old, new))
    subprocess.run(["gcc", *CFLAGS, path_c, "-o", path_so, "-lm"], check=True, capture_output=True)
    return name, _run_pins(path_so).returncode == 0


def test_every_planted_mistake_fails_a_pin(tmp_path):
    # the unmodified oracle, run the same way, passes
    import oracle
    assert _run_pins(oracle.build()).returncode == 0
    jobs = [(n, o, r, str(tmp_path)) for n, o, r in MUTANTS]
    with ThreadPoolExecutor(max_workers=max(2, (os.cpu_count() or 2) // 2)) as pool:
        results = list(pool.map(_mutant_survives, jobs))
    survivors = [n for n, alive in results if alive]
    assert not survivors, f"pins did not notice: {survivors}"
