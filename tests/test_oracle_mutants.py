"""The pins must notice a wrong oracle: each case plants one plausible mistake in a copy of
oracle.cpp (on the CPU, in a temporary directory), rebuilds it, and expects the pin suite to fail."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SOURCE = os.path.join(ROOT, "oracle", "oracle.cpp")

MUTANTS = {
    "gcn_tolerance_scale_inflated": ("                    aabs += std::fabs(m);\n                }\n                out[r * f + j] = acc;\n                if (abs_out) abs_out[r * f + j] = aabs;\n            }\n        }\n    }\n    return 0;\n}\n\n// GAT attention scores",
                                     "                    aabs += 2.0 * std::fabs(m);\n                }\n                out[r * f + j] = acc;\n                if (abs_out) abs_out[r * f + j] = aabs;\n            }\n        }\n    }\n    return 0;\n}\n\n// GAT attention scores"),
    "gat_tolerance_scale_inflated": ("                    const double m = a[k - b] * load_x(z, zdt, (int64_t)col_idx[k] * ldz + j);\n                    acc += m;\n                    aabs += std::fabs(m);",
                                     "                    const double m = a[k - b] * load_x(z, zdt, (int64_t)col_idx[k] * ldz + j);\n                    acc += m;\n                    aabs += 100.0 * std::fabs(m);"),
    "gat_tolerance_scale_runs_on_across_columns": ("                double acc = 0.0, aabs = 0.0;\n                for (int32_t k = b; k < e; ++k) {\n                    const double m = a[k - b]",
                                                   "                double acc = 0.0; static thread_local double aabs = 0.0;\n                for (int32_t k = b; k < e; ++k) {\n                    const double m = a[k - b]"),
    "fp32_score_wrapper_swaps_source_and_destination": ("return orc_edge_softmax(n, row_ptr, col_idx, a.data(), b.data(), heads, slope, alpha);",
                                                        "return orc_edge_softmax(n, row_ptr, col_idx, b.data(), a.data(), heads, slope, alpha);"),
    "fp32_score_wrapper_reuses_source_scores": ("for (size_t i = 0; i < a.size(); ++i) { a[i] = s_src[i]; b[i] = s_dst[i]; }",
                                                "for (size_t i = 0; i < a.size(); ++i) { a[i] = s_src[i]; b[i] = s_src[i]; }"),
    "gcn_weight_uses_destination_twice": ("const double w = model == 0 ? dinv[u] * dinv[v] : rdeg;",
                                          "const double w = model == 0 ? dinv[v] * dinv[v] : rdeg;"),
    "csr_rows_by_source": ("edges.push_back({d, s, i});", "edges.push_back({s, d, i});"),
    "leaky_slope_dropped": ("a[k - b] = t >= 0.0 ? t : slope * t;", "a[k - b] = t;"),
    "attention_vectors_swapped": ("ss += (double)a_src[h * dim + d] * zv;", "ss += (double)a_dst[h * dim + d] * zv;"),
    "softmax_without_max_is_fine_but_sum_misses_last": (
        "for (int32_t k = b; k < e; ++k) { a[k - b] = std::exp(a[k - b] - mx); sum += a[k - b]; }",
        "for (int32_t k = b; k < e; ++k) { a[k - b] = std::exp(a[k - b] - mx); if (k + 1 < e || e - b == 1) sum += a[k - b]; }"),
    "self_loops_not_replaced": ("edges.erase(std::remove_if(edges.begin(), edges.end(), [](const Edge& x) { return x.src == x.dst; }),\n                    edges.end());", ""),
    "dedup_keeps_last": ("if (a.src != b.src) return a.src < b.src;\n        return a.id < b.id;",
                         "if (a.src != b.src) return a.src < b.src;\n        return a.id > b.id;"),
    "mean_divides_by_degree_plus_one": ("const double rdeg = e > b ? 1.0 / (double)(e - b) : 0.0;",
                                        "const double rdeg = e > b ? 1.0 / (double)(e - b + 1) : 0.0;"),
    "last_chunk_column_dropped": ("const int32_t j0 = p * chunk_width, j1 = std::min(f, j0 + chunk_width);\n#pragma omp parallel for schedule(dynamic, 64) num_threads(threads > 1 ? threads : 1) if (threads > 1)\n        for (int64_t r = 0; r < count; ++r) {\n            const int64_t v = rows ? rows[r] : r;\n            const int32_t b = row_ptr[v], e = row_ptr[v + 1];\n            const double rdeg",
                                  "const int32_t j0 = p * chunk_width, j1 = std::min(f - (p > 0 ? 1 : 0), j0 + chunk_width);\n#pragma omp parallel for schedule(dynamic, 64) num_threads(threads > 1 ? threads : 1) if (threads > 1)\n        for (int64_t r = 0; r < count; ++r) {\n            const int64_t v = rows ? rows[r] : r;\n            const int32_t b = row_ptr[v], e = row_ptr[v + 1];\n            const double rdeg"),
}


def run_pins(tmp_path, source_text):
    src = tmp_path / "oracle_mutant.cpp"
    src.write_text(source_text)
    env = dict(os.environ, GNNFD_ORACLE_SOURCE=str(src), GNNFD_ORACLE_LIB=str(tmp_path / "liboracle_mutant.so"),
               PYTHONPATH=ROOT)
    return subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_oracle_pins.py"), "-x", "-q",
                           "-p", "no:cacheprovider"], env=env, cwd=ROOT, capture_output=True, text=True)


def test_unmodified_copy_passes(tmp_path):
    res = run_pins(tmp_path, open(SOURCE).read())
    assert res.returncode == 0, res.stdout[-2000:]


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_pins_reject_mutant(tmp_path, name):
    old, new = MUTANTS[name]
    text = open(SOURCE).read()
    assert text.count(old) >= 1, "mutation site not found: %s" % name
    res = run_pins(tmp_path, text.replace(old, new, 1))
    assert res.returncode != 0, "the pins accepted the mutant '%s'" % name
