"""Are the oracle's pins strong enough?  Each case plants one plausible mistake in a COPY of the
oracle's source (a dropped term, a wrong index, a swapped order, a wrong tie rule), compiles it, and
runs the pin tests against the broken library: they must fail.  CPU only; the real oracle is
never modified."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "slonn_oracle.c")

MUTANTS = {
    "partial index ignores the chunk width": ("uint32_t p = (uint32_t)((j / V) % 32u);", "uint32_t p = (uint32_t)(j % 32u);"),
    "tree adds neighbours first": ("for (int off = 16; off >= 1; off >>= 1)\n        for (int p = 0; p < off; ++p) acc[p] = acc[p] + acc[p + off];",
                                   "for (int off = 1; off <= 16; off <<= 1)\n        for (int p = 0; p + off < 32; p += 2 * off) acc[p] = acc[p] + acc[p + off];"),
    "bias dropped": ("return acc[0] + bias;", "return acc[0];"),
    "budget rounds down": ("((uint64_t)bp * N + 5000u) / 10000u", "((uint64_t)bp * N) / 10000u"),
    "ranking ascending": ("if (sa > sb) return -1;\n    if (sa < sb) return 1;", "if (sa > sb) return 1;\n    if (sa < sb) return -1;"),
    "ties by higher id": ("return (a < b) ? -1 : (a > b) ? 1 : 0;", "return (a < b) ? 1 : (a > b) ? -1 : 0;"),
    "key bits reversed at run time": ("if (bit) key |= (1u << j);", "if (bit) key |= (1u << (m->K - 1u - j));"),
    "lists read table by table": ("for (uint32_t r = 0; r < cap && got < B; ++r)\n        for (uint32_t b = 0; b < L && got < B; ++b) {",
                                  "for (uint32_t b = 0; b < L && got < B; ++b)\n        for (uint32_t r = 0; r < cap && got < B; ++r) {"),
    "hidden activation not rectified": ("return z > 0.0f ? z : 0.0f;", "return z;"),
    "sample variance instead of population variance": ("for (uint32_t i = 0; i < N; ++i) var[i] = var[i] / (double)n_cal;",
                                                       "for (uint32_t i = 0; i < N; ++i) var[i] = var[i] / (double)(n_cal - 1);"),
    "empty buckets get the identity order": ("{ sort_ctx c = { global }; qsort_r(glist, N, sizeof(uint32_t), cmp_rank, &c); }", "{ }"),
    "free variant: hash nodes stay in the lists": ("if (!is_hash[src[i]]) dst[o++] = src[i];", "dst[o++] = src[i];"),
    "free variant: hash nodes missing from the active set": ("for (uint32_t h = 0; h < H; ++h) seen[m->hash_nodes[l][h]] = 1;\n    if (want", "if (want"),
    "free variant: the budget counts the hash nodes": ("const uint32_t want = B < N - H ? B : N - H;", "const uint32_t want = B > H ? (B - H < N - H ? B - H : N - H) : 0;"),
    "generator constant mistyped": ("0xBF58476D1CE4E5B9ull", "0xBF58476D1CE4E5B1ull"),
    "hash bit of zero counts as set": ("node_z32_dense(m, l, h, in32)) > 0.0f;", "node_z32_dense(m, l, h, in32)) >= 0.0f;"),
    "scores summed in fp32": ("for (uint32_t i = 0; i < N; ++i) s[i] += (double)a[i];", "for (uint32_t i = 0; i < N; ++i) s[i] = (double)((float)s[i] + a[i]);"),
    "LCAO takes the smallest feasible budget": ("(!found || profile_bp[i] > best)", "(!found || profile_bp[i] < best)"),
    "LCAO ignores the time already spent": ("if (t0[q] + profile_ms[i] <= tau[q]", "if (profile_ms[i] <= tau[q]"),
    "confidence: log-sum-exp forgets the shift": ("const double lse_k = mk + log(sk);", "const double lse_k = log(sk);"),
    "confidence: the k% prediction is the target": ("const double y = exp((double)z_full[j] - mf) / sf;\n        c += y * ((double)z_k[j] - lse_k);",
                                                    "const double y = exp((double)z_k[j] - mk) / sk;\n        c += y * ((double)z_full[j] - mf - log(sf));"),
    "confidence tables: counts keyed by the last activator": ("count[b * nb + codes[((uint64_t)x * n_act + 0) * L + b]] += 1;",
                                                              "count[b * nb + codes[((uint64_t)x * n_act + n_act - 1) * L + b]] += 1;"),
    "ACLO takes the largest k that meets its threshold": ("if (!ok && rows && est >= (double)thr[i])", "if (rows && est >= (double)thr[i])"),
    "ACLO threshold strict": ("est >= (double)thr[i]", "est > (double)thr[i]"),
    "ACLO estimate averages per-table means": ("const double est = rows ? s / (double)rows : 0.0;",
                                               "double est = 0.0; for (uint32_t b = 0; b < L; ++b) if (count[b * nb + keys[b]]) est += sum[((uint64_t)b * nb + keys[b]) * n_k + i] / count[b * nb + keys[b]] / L; (void)s;"),
    "argmax keeps the last maximum": ("if (ref ? (out64[n] > out64[best]) : (out32[n] > out32[best])) best = n;",
                                      "if (ref ? (out64[n] >= out64[best]) : (out32[n] >= out32[best])) best = n;"),
}


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_pins_catch_planted_mistake(name, tmp_path):
    old, new = MUTANTS[name]
    text = open(SRC).read()
    assert text.count(old) >= 1, f"mutation site for '{name}' not found: the oracle's source changed"
    src = tmp_path / "mutant.c"
    src.write_text(text.replace(old, new, 1))
    lib = tmp_path / "libmutant.so"
    subprocess.run(["gcc", "-O1", "-std=c11", "-D_GNU_SOURCE", "-ffp-contract=off", "-mfma", "-fopenmp", "-fPIC", "-shared",
                    "-o", str(lib), str(src), "-lm"], check=True)
    env = dict(os.environ, SLONN_ORACLE_LIB=str(lib), OMP_NUM_THREADS="2")
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                        os.path.join(ROOT, "tests", "test_oracle_pins.py"), os.path.join(ROOT, "tests", "test_oracle_method.py"),
                        os.path.join(ROOT, "tests", "test_lcao.py"), os.path.join(ROOT, "tests", "test_oracle_free_hash.py"),
                        os.path.join(ROOT, "tests", "test_aclo.py"),
                        "-m", "not gpu"],
                       env=env, cwd=ROOT, capture_output=True, text=True)
    assert r.returncode == 1, f"the pins did not notice: {name}\n{r.stdout[-600:]}"
