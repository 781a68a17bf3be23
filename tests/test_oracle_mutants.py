"""Do the pins bite?  Each case plants one plausible mistake in a COPY of the CPU checker's source (a dropped term,
a wrong sign or index, a transposed operand, a wrong rounding or ordering rule), builds it, and runs the pins that
are meant to catch that kind of mistake against the broken build: they must fail.  The mistakes are planted in the
checker, on the CPU; nothing here touches a GPU or the CUDA library."""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "dg4_oracle.cpp")

# (name, text in the checker's source, what replaces it, -k expression selecting the pins expected to object)
MUTANTS = [
    ("level_without_plus_one", "lv = std::max(lv, level[u] + 1);", "lv = std::max(lv, level[u]);",
     "levels or fixture or generated"),
    ("cone_one_hop_short", "for (int step = 0; step < hops; ++step) {", "for (int step = 0; step + 1 < hops; ++step) {",
     "cones or fixture or neighbourhood or binary"),
    ("cone_without_self", "total += 1 + (int64_t)cone.size();", "total += (int64_t)cone.size();",
     "cones or fixture or neighbourhood or binary"),
    ("cone_only_last_frontier", "for (int u : next) cone.insert(u);", "cone = next;",
     "cones or fixture or neighbourhood or binary"),
    ("buckets_descending", "return level[a] < level[b]; });", "return level[a] > level[b]; });", "bucket or level"),
    ("class_order_ties_by_descending_id", "            return a < b;\n        });", "            return a > b;\n        });",
     "class"),
    ("partition_stride_off_by_one", "(level[v] - k) % delta == 0;", "(level[v] - k) % (delta + 1) == 0;", "partition"),
    ("partition_stride_from_level_zero", "level[v] >= k && (level[v] - k) % delta == 0;", "level[v] % delta == 0;",
     "partition"),
    ("partition_forgets_fanout_free_nodes", "if (on_stride_level || !has_fanout[v]) picked.push_back(v);",
     "if (on_stride_level) picked.push_back(v);", "partition"),
    ("partition_groups_count_inclusive", "below += (level[v] < l);", "below += (level[v] <= l);", "partition"),
    ("score_without_scale", "s[j] = scale * dot;", "s[j] = dot;", "attention or closed or dense"),
    ("score_sign", "s[j] = scale * dot;", "s[j] = -scale * dot;", "attention or closed or dense"),
    ("softmax_not_normalised", "for (int j = 0; j < cnt; ++j) a[j] /= z;\n    for (int c = 0; c < d_head; ++c) {",
     "for (int c = 0; c < d_head; ++c) {", "attention or closed or sum"),
    ("head_slices_of_key_ignored", "kr[j] = K + u * d + h * dh;", "kr[j] = K + u * d;", "attention or dense or heads"),
    ("value_of_the_destination", "vr[j] = V + u * d + h * dh;", "vr[j] = V + (int64_t)v * d + h * dh;",
     "attention or closed or dense"),
    ("additive_without_leaky_slope", "e[j] = x > 0.0 ? x : slope * x;", "e[j] = x;", "additive"),
    ("projection_transposed", "acc += x[c] * W[(int64_t)o * d_in + c];", "acc += x[c] * W[(int64_t)c * d_out + o];",
     "project or layer"),
    ("projection_without_residual", "if (r) acc += r[o];", "", "project or layer or residual"),
    ("levelised_in_reverse_order", "for (int l = 0; l < n_levels; ++l) {\n        int lo = level_ptr[l], hi = level_ptr[l + 1];",
     "for (int l = n_levels - 1; l >= 0; --l) {\n        int lo = level_ptr[l], hi = level_ptr[l + 1];", "levelised"),
    ("bf16_by_truncation", "double r = std::nearbyint(x / q) * q;", "double r = std::trunc(x / q) * q;", "bf16 or rounding"),
    ("layernorm_unbiased_variance", "        var /= d;\n", "        var /= (d - 1);\n", "layernorm or ffn"),
    ("layernorm_eps_outside_root", "double rstd = 1.0 / std::sqrt(var + eps);", "double rstd = 1.0 / (std::sqrt(var) + eps);",
     "layernorm or ffn"),
    ("layernorm_gamma_beta_swapped", "(x[c] - mean) * rstd * gamma[c] + beta[c];", "(x[c] - mean) * rstd * beta[c] + gamma[c];",
     "layernorm or ffn"),
    ("ffn_without_first_bias", "double acc = b1[h];", "double acc = 0.0;", "ffn"),
    ("ffn_without_relu", "acc = acc > 0.0 ? acc : 0.0;", "", "ffn"),
    ("ffn_without_residual", "z[o] = x[o] + acc;", "z[o] = acc;", "ffn"),
    ("update_frozen_gate_stored_again", "                if (!updated[v]) {\n                    std::memcpy(hist", "                if (true) {\n                    std::memcpy(hist", "cone_update"),
    ("update_frozen_gate_keeps_in_edges", "                if (!updated[v])\n                    for (int e = cone_ptr[v] + 1;", "                if (true)\n                    for (int e = cone_ptr[v] + 1;", "cone_update"),
    ("update_marks_only_the_stored_gates", "            for (int v : S) updated[v] = 1;", "            for (int r = b0; r < b1; ++r) updated[roots[r]] = 1;", "cone_update"),
    ("update_inputs_not_from_the_table", "std::memcpy(&cur[(int64_t)i * d], hist + (int64_t)S[i] * d, sizeof(double) * d);",
     "std::memcpy(&cur[(int64_t)i * d], X + (int64_t)S[i] * d, sizeof(double) * d);", "cone_update"),
    ("update_one_layer_only", "            for (int j = 0; j < n_layers; ++j) {\n                orc_layer_parallel(m,", "            for (int j = 0; j < 1; ++j) {\n                orc_layer_parallel(m,", "cone_update"),
    ("update_batches_span_level_groups", "const int b1 = std::min(b0 + batch, (int)group_ptr[l + 1]);", "const int b1 = std::min(b0 + batch, (int)group_ptr[n_levels]);", "cone_update"),
    ("block_levelised_in_reverse_order", "for (int lev = 0; lev < n_levels; ++lev) {", "for (int lev = n_levels - 1; lev >= 0; --lev) {", "block_levelised"),
    ("block_levelised_skips_first_norm", "            orc_layernorm(1, d, pre.data(), g1, be1, eps, h1.data());", "            h1 = pre;", "block_levelised"),
    ("block_levelised_keys_from_attention_sublayer_output", "orc_ffn(1, d, d_ff, h1.data(), W1, b1, W2, b2, g2, be2, eps, rounding, fresh.data() + (int64_t)(i - lo) * d);",
     "std::memcpy(fresh.data() + (int64_t)(i - lo) * d, h1.data(), sizeof(double) * d);", "block_levelised"),
    ("block_levelised_without_attention_residual", "project_row(d, d, o.data(), W_o, H + (int64_t)v * d, pre.data());",
     "project_row(d, d, o.data(), W_o, nullptr, pre.data());", "block_levelised"),
    ("ffn_second_matrix_transposed", "acc += u[h] * W2[(int64_t)o * d_ff + h];", "acc += u[h] * W2[(int64_t)h * d + o];", "ffn"),
]


def _run_mutant(args):
    source, tmp, name, old, new, pins = args
    if source.count(old) != 1:
        return name, f"the text to replace must occur exactly once ({source.count(old)} times)"
    src = os.path.join(tmp, name + ".cpp")
    with open(src, "w") as f:
        f.write(source.replace(old, new))
    lib = os.path.join(tmp, name + ".so")
    subprocess.check_call(["g++", "-O1", "-fopenmp", "-shared", "-fPIC", "-w", "-o", lib, src])
    env = dict(os.environ, DG4_ORACLE_LIB=lib, OMP_NUM_THREADS="2")
    run = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_oracle_pins.py"),
                          os.path.join(ROOT, "tests", "test_oracle_cone_update.py"), "-x", "-q",
                          "-p", "no:cacheprovider", "-k", pins], cwd=ROOT, env=env, capture_output=True, text=True)
    if run.returncode != 1:          # 1 = some selected pin failed; 0 = all passed; 5 = none selected
        return name, f"pytest exit code {run.returncode}:\n{run.stdout[-1500:]}"
    return name, None


def test_pins_reject_every_planted_mistake(tmp_path):
    source = open(SRC).read()
    jobs = [(source, str(tmp_path), *m) for m in MUTANTS]
    with ThreadPoolExecutor(max_workers=max(1, min(8, (os.cpu_count() or 2) // 2))) as pool:
        results = list(pool.map(_run_mutant, jobs))
    survivors = [(name, why) for name, why in results if why is not None]
    assert not survivors, "the pins did not object to: " + "; ".join(f"{n} ({w})" for n, w in survivors)
