"""Do the pins notice a mistake?  Each case plants ONE plausible mistake in a copy of the oracle's source
(never in the CUDA path), builds it, and runs the oracle's pin tests against that build in a child process:
at least one pin must fail.  The unchanged copy must pass.  The children run side by side."""
import os
import subprocess
import sys

import pytest

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
SRC = os.path.join(ROOT, "oracle", "pyramidkv_oracle.cpp")
PINS = ["test_oracle_budgets.py", "test_oracle_scores.py", "test_oracle_select_gather.py", "test_oracle_dtypes.py",
        "test_oracle_paged.py", "test_oracle_planted.py"]

# (name, text in the oracle, replacement[, which occurrence when the text appears more than once])
MUTANTS = [
    ("control", None, None),
    ("mask_off_by_one", "const int visible = P + j + 1;", "const int visible = P + j;"),
    ("mask_not_causal", "const int visible = P + j + 1;", "const int visible = n;"),
    ("no_scale", "logit[i] = dot * scale;", "logit[i] = dot;"),
    ("scale_by_d", "const double scale = 1.0 / std::sqrt(static_cast<double>(d));",
     "const double scale = 1.0 / static_cast<double>(d);", 0),
    ("decode_scale_by_d", "const double scale = 1.0 / std::sqrt(static_cast<double>(d));",
     "const double scale = 1.0 / static_cast<double>(d);", 2),
    ("sum_over_group_not_mean", "const double inv_group = 1.0 / static_cast<double>(group);",
     "const double inv_group = 1.0;"),
    ("max_subtraction_dropped", "logit[i] = std::exp(logit[i] - mx);", "logit[i] = std::exp(logit[i]);"),
    ("lse_without_max", "row_lse[static_cast<int64_t>(hq) * alpha + j] = mx + std::log(z);",
     "row_lse[static_cast<int64_t>(hq) * alpha + j] = std::log(z);"),
    ("wrong_query_head", "const int hq = h * group + g;", "const int hq = g * num_kv_heads + h;"),
    ("pool_radius", "const int r = (w - 1) / 2;\n  for (int i = 0; i < P; ++i) {\n    float best = in[i];",
     "const int r = w / 2 + 1;\n  for (int i = 0; i < P; ++i) {\n    float best = in[i];"),
    ("pool_one_sided", "for (int t = -r; t <= r; ++t) {\n      const int x = i + t;\n      if (x >= 0 && x < P) best",
     "for (int t = 0; t <= r; ++t) {\n      const int x = i + t;\n      if (x >= 0 && x < P) best"),
    ("avg_pool_divides_by_count", "out[i] = sum / static_cast<float>(w);",
     "out[i] = sum / static_cast<float>(std::min(P - 1, i + r) - std::max(0, i - r) + 1);"),
    ("sort_ascending", "return pooled[a] > pooled[b];", "return pooled[a] < pooled[b];"),
    ("leftover_to_top_layers", "for (int l = 0; l < m && left > 0; ++l, --left) k_out[l] += 1;",
     "for (int l = m - 1; l >= 0 && left > 0; --l, --left) k_out[l] += 1;", 0),
    ("geometric_leftover_to_top_layers", "for (int l = 0; l < m && left > 0; ++l, --left) k_out[l] += 1;",
     "for (int l = m - 1; l >= 0 && left > 0; --l, --left) k_out[l] += 1;", 1),
    ("pyramid_over_whole_budget", "const int64_t k_total = static_cast<int64_t>(m) * (avg_budget - alpha);",
     "const int64_t k_total = static_cast<int64_t>(m) * avg_budget;", 0),
    ("geometric_over_whole_budget", "const int64_t k_total = static_cast<int64_t>(m) * (avg_budget - alpha);",
     "const int64_t k_total = static_cast<int64_t>(m) * avg_budget;", 1),
    ("geometric_grows_with_depth", "power[m - 1 - l] / total", "power[l] / total"),
    ("geometric_top_layer_rule", "static_cast<double>(bq) / 1024.0 * m;", "static_cast<double>(bq) / 1024.0;"),
    ("geometric_ratio_not_snapped", "rho = std::round(0.5 * (lo + hi) * 1048576.0) / 1048576.0;",
     "rho = std::round(0.5 * (lo + hi) * 1024.0) / 1024.0;"),
    ("slope_sign", "static_cast<__int128>(2 * bq - 2048) * l;", "static_cast<__int128>(2048 - 2 * bq) * l;"),
    ("short_context_still_compressed", "if (n <= avg_budget) return n;", "if (n <= alpha) return n;"),
    ("window_dropped", "for (int i = P; i < n; ++i) row[cnt++] = i;", "for (int i = P; i < n; ++i) row[cnt++] = P;"),
    ("v_copied_from_k", "static_cast<const char*>(v) + src, d * esz);", "static_cast<const char*>(k) + src, d * esz);"),
    ("fp16_bias", "e - 15);", "e - 16);"),
    ("attention_mask_off_by_one", "if (pos[r] > P + j) {", "if (pos[r] >= P + j) {"),
    ("attention_not_normalised", "o += (w[r] / z) * elem(vc,", "o += w[r] * elem(vc,", 0),
    ("attention_values_from_k", "o += (w[r] / z) * elem(vc,", "o += (w[r] / z) * elem(kc,", 0),
    ("attention_no_scale", "w[r] = dot * scale;\n      mx = std::max(mx, w[r]);\n    }\n    double z = 0.0;\n    for (int r = 0; r < c; ++r) { w[r] = std::exp(w[r] - mx); z += w[r]; }\n    for (int t = 0; t < d; ++t) {\n      double o = 0.0;",
     "w[r] = dot;\n      mx = std::max(mx, w[r]);\n    }\n    double z = 0.0;\n    for (int r = 0; r < c; ++r) { w[r] = std::exp(w[r] - mx); z += w[r]; }\n    for (int t = 0; t < d; ++t) {\n      double o = 0.0;"),
    ("page_slot", "* page_size + (r % page_size)) * row_bytes;\n    std::memcpy(static_cast<char*>(pool) + dst",
     "* page_size + (r / page_size)) * row_bytes;\n    std::memcpy(static_cast<char*>(pool) + dst"),
]


def test_every_planted_mistake_fails_a_pin(tmp_path):
    source = open(SRC).read()
    children = []
    for name, old, new, *which in MUTANTS:
        text = source
        if old is not None:
            places = [i for i in range(len(source)) if source.startswith(old, i)]
            assert places and (which or len(places) == 1), "mutation point of %s: %d places" % (name, len(places))
            at = places[which[0] if which else 0]
            text = source[:at] + new + source[at + len(old):]
        cpp = tmp_path / ("%s.cpp" % name)
        lib = tmp_path / ("lib_%s.so" % name)
        cpp.write_text(text)
        subprocess.check_call(["g++", "-O1", "-std=c++17", "-fopenmp", "-fPIC", "-shared", "-o", str(lib), str(cpp)])
        env = dict(os.environ, PKV_ORACLE_LIB=str(lib), OMP_NUM_THREADS="1", MKL_NUM_THREADS="1")
        cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider", "-m", "not gpu"] + \
              [os.path.join(HERE, f) for f in PINS]
        children.append((name, subprocess.Popen(cmd, cwd=ROOT, env=env, stdout=subprocess.PIPE,
                                                stderr=subprocess.STDOUT, text=True)))
    survivors, control = [], None
    for name, proc in children:
        out, _ = proc.communicate(timeout=900)
        if name == "control":
            control = (proc.returncode, out[-2000:])
        elif proc.returncode == 0:
            survivors.append(name)
        else:
            assert " failed" in out and "error" not in out.splitlines()[-1], "%s: the run broke:\n%s" % (name, out[-1500:])
    assert control[0] == 0, "the unchanged oracle fails its own pins:\n" + control[1]
    assert not survivors, "no pin noticed: %s" % ", ".join(survivors)
