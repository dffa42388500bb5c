"""Do the pins have teeth? Each case plants one plausible mistake in a copy of the CPU oracle (a wrong sign,
an off-by-one, a swapped operand, a dropped factor), compiles the copy, and runs the pin files that cover the
mutated part against it in a child pytest: at least one pin must fail. The unmutated source is also run through
the same machinery and must pass, so a failure here is never the machinery's own.

Everything happens on the CPU, in copies under a temporary directory; the in-tree oracle is not touched."""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SOURCE = os.path.join(ROOT, "oracle", "swarm_oracle.cpp")

# (name, text in the oracle source, replacement, pin files that must notice)
MUTANTS = [
    ("philox_mixes_the_wrong_product", "const uint32_t n0 = hi1 ^ c1 ^ k0;", "const uint32_t n0 = hi0 ^ c1 ^ k0;",
     ["test_oracle_rng.py"]),
    ("philox_key_schedule_starts_a_round_early", "if (round > 0) { k0 += kWeyl0; k1 += kWeyl1; }",
     "{ k0 += kWeyl0; k1 += kWeyl1; }", ["test_oracle_rng.py"]),
    ("box_muller_radius_without_the_factor_two", "std::sqrt(-2.0 * std::log(u1))", "std::sqrt(-1.0 * std::log(u1))",
     ["test_oracle_rng.py"]),
    ("uniform_float_drops_a_bit", "return (float)(word >> 8) * 0x1p-24f;", "return (float)(word >> 9) * 0x1p-24f;",
     ["test_oracle_rng.py"]),
    ("uniform_int_takes_the_low_half", "return (uint32_t)(((uint64_t)word * m) >> 32);",
     "return (uint32_t)(((uint64_t)word * m) & 0xFFFFFFFFu) % m;", ["test_oracle_rng.py"]),
    ("exponent_rule_not_least_at_equality", "while ((double)L * std::ldexp(1.0, e) < (double)rho) ++e;",
     "while ((double)L * std::ldexp(1.0, e) <= (double)rho) ++e;", ["test_oracle_quantizer.py"]),
    ("rounding_threshold_inclusive", "return (int32_t)((uint32_t)base + (u16 < thr ? 1u : 0u));",
     "return (int32_t)((uint32_t)base + (u16 <= thr ? 1u : 0u));", ["test_oracle_quantizer.py"]),
    ("rounding_always_down", "return (int32_t)((uint32_t)base + (u16 < thr ? 1u : 0u));",
     "return (int32_t)((uint32_t)base);", ["test_oracle_quantizer.py", "test_oracle_interact.py"]),
    ("decode_window_shifted_by_one", "if (delta > (1 << (bits - 1))) delta -= (1 << bits);",
     "if (delta >= (1 << (bits - 1))) delta -= (1 << bits);", ["test_oracle_quantizer.py"]),
    ("packing_big_endian_bits", "block_bytes[pos / 8] = (uint8_t)(block_bytes[pos / 8] | (1u << (pos % 8)));",
     "block_bytes[pos / 8] = (uint8_t)(block_bytes[pos / 8] | (1u << (7 - pos % 8)));", ["test_oracle_quantizer.py"]),
    ("bf16_rounds_half_up", "u += 0x7FFFu + lsb;", "u += 0x8000u;", ["test_oracle_quantizer.py"]),
    ("plain_average_keeps_one_model", "const float v = 0.5f * (xa[k] + xb[k]); xa[k] = v; xb[k] = v;",
     "const float v = 0.5f * (xa[k] + xb[k]); xa[k] = v;", ["test_oracle_interact.py"]),
    ("quantized_average_has_a_sign_slip", "const float v = 0.5f * (Qa + Qb);", "const float v = 0.5f * (Qa - Qb);",
     ["test_oracle_interact.py"]),
    ("blocking_decode_with_a_doubled_step", "const float Qa = dec(xb[k0 + k], get_code(ca, k, bits), e, bits);",
     "const float Qa = dec(xb[k0 + k], get_code(ca, k, bits), e + 1, bits);", ["test_oracle_interact.py"]),
    ("blocking_range_ignores_one_model", "rho = std::max(rho, std::fabs(va - vb));\n      M = std::max(M, std::max(std::fabs(va), std::fabs(vb)));",
     "rho = std::max(rho, std::fabs(va));\n      M = std::max(M, std::max(std::fabs(va), std::fabs(vb)));",
     ["test_oracle_interact.py"]),
    ("nonblocking_pending_update_added", "const float nx = av - D;\n      avg[k] = av; new_x[k] = nx;\n      spread = std::max(spread, std::fabs(own - oth));",
     "const float nx = av + D;\n      avg[k] = av; new_x[k] = nx;\n      spread = std::max(spread, std::fabs(own - oth));",
     ["test_oracle_interact.py"]),
    ("nonblocking_touches_the_responder", "for (int k = 0; k < len; ++k) { xa[k0 + k] = new_x[k]; ba[k0 + k] = new_x[k]; }\n  }\n  s.w[a] += 1; s.w[b] += 1;\n}",
     "for (int k = 0; k < len; ++k) { xa[k0 + k] = new_x[k]; ba[k0 + k] = new_x[k]; s.x(b)[k0 + k] = avg[k]; }\n  }\n  s.w[a] += 1; s.w[b] += 1;\n}",
     ["test_oracle_interact.py"]),
    ("register_chain_uses_the_wrong_key", "const float Qb = dec(qhat_b[k], get_code(cb, k, bits), epb, bits);",
     "const float Qb = dec(qhat_a, get_code(cb, k, bits), epb, bits);", ["test_oracle_registers.py"]),
    ("register_update_sign", "const float nx = av - D;\n      avg[k] = av; new_x[k] = nx;\n      spread = std::max(spread, std::fabs(Qa - Qb));",
     "const float nx = av + D;\n      avg[k] = av; new_x[k] = nx;\n      spread = std::max(spread, std::fabs(Qa - Qb));",
     ["test_oracle_registers.py"]),
    ("every_reader_gets_the_first_readers_prefix", "bits, prefixes ? prefixes[p] : s.own_prefix);",
     "bits, prefixes ? prefixes[0] : s.own_prefix);", ["test_oracle_registers.py"]),
    ("clock_of_the_initiator_not_reset", "s.tau[pairs[2 * p]] = 0;", "s.tau[pairs[2 * p + 1]] = 0;",
     ["test_oracle_registers.py", "test_oracle_graph.py", "test_oracle_staleness.py"]),
    ("lsq_gradient_not_averaged_over_the_batch", "g /= (double)bsz;", "", ["test_oracle_local_steps.py"]),
    ("lsq_residual_sign", "resid[t] = pred - (double)s.bvec[(size_t)i * m + rows[t]];",
     "resid[t] = pred + (double)s.bvec[(size_t)i * m + rows[t]];", ["test_oracle_local_steps.py"]),
    ("lsq_steps_all_at_the_first_iterate", "minibatch_rows(s, i, s.ls[i], rows.data());",
     "minibatch_rows(s, i, 0, rows.data());", ["test_oracle_local_steps.py"]),
    ("synthetic_step_ascends", "xi[k] = xi[k] - st;", "xi[k] = xi[k] + st;", ["test_oracle_local_steps.py"]),
    ("geometric_count_off_by_one", "if (uniform_int(wd[t % 4], (uint32_t)mean_h) == 0) return t + 1;",
     "if (uniform_int(wd[t % 4], (uint32_t)mean_h) == 0) return t;", ["test_oracle_local_steps.py"]),
    ("sampler_reuses_one_word", "const int j = s.adj[(size_t)i * s.degree + uniform_int(wd[1], (uint32_t)s.degree)];",
     "const int j = s.adj[(size_t)i * s.degree + uniform_int(wd[0], (uint32_t)s.degree)];", ["test_oracle_graph.py"]),
    ("sampler_allows_shared_nodes", "if (used[i] || used[j]) continue;", "if (used[i]) continue;", ["test_oracle_graph.py"]),
    ("regular_graph_one_directional", "edge[(size_t)u * n + v] = edge[(size_t)v * n + u] = 1;", "edge[(size_t)u * n + v] = 1;",
     ["test_oracle_graph.py"]),
    ("potential_around_the_wrong_centre", "mu /= (double)s.n;\n    for (int i = 0; i < s.n; ++i) { const double t = (double)s.x(i)[k] - mu; gamma += t * t; }",
     "mu /= (double)(s.n + 1);\n    for (int i = 0; i < s.n; ++i) { const double t = (double)s.x(i)[k] - mu; gamma += t * t; }",
     ["test_oracle_interact.py"]),
    ("mean_model_is_a_sum", "out[k] = (float)(acc / (double)s.n);", "out[k] = (float)(acc);",
     ["test_oracle_interact.py", "test_oracle_staleness.py"]),
    ("guard_distance_counts_the_spread_once", "const float rho = 2.0f * spread + dmax;\n    const int e = exponent_rule(rho, M, bits);",
     "const float rho = spread + dmax;\n    const int e = exponent_rule(rho, M, bits);", ["test_oracle_interact.py"]),
    ("one_way_write_scaled_by_the_new_model_alone", "M = std::max(M, std::max(std::fabs(nx), std::fabs(av)));\n    }\n    const float rho = 2.0f * spread + dmax;\n    const int e = exponent_rule(rho, M, bits);",
     "M = std::max(M, std::fabs(nx));\n    }\n    const float rho = 2.0f * spread + dmax;\n    const int e = exponent_rule(rho, M, bits);",
     ["test_oracle_interact.py"]),
    ("responder_register_scaled_to_the_wrong_key", "write_current_block(s, b, blk, avg.data(), qhat_b.data(), len, bits);",
     "write_current_block(s, b, blk, avg.data(), qhat_new.data(), len, bits);", ["test_oracle_registers.py"]),
    ("own_register_resolution_follows_the_code_width", "const int eo = exponent_rule(rho, M, kOwnResolutionBits);\n    write_own_block(s, a,",
     "const int eo = exponent_rule(rho, M, bits);\n    write_own_block(s, a,", ["test_oracle_registers.py"]),
    ("rounding_uniform_halves_swapped", "return (k % 2 == 0) ? (word & 0xFFFFu) : (word >> 16);\n}\n\n// Packing",
     "return (k % 2 == 1) ? (word & 0xFFFFu) : (word >> 16);\n}\n\n// Packing", ["test_oracle_rng.py"]),
    ("initial_models_without_the_node_offset", "xi[k] = p + s.offset[i];", "xi[k] = p;", ["test_oracle_rng.py", "test_oracle_interact.py"]),
    ("labels_without_the_node_shift", "const float score = (float)(acc + (double)s.shift[i] + (double)noise);",
     "const float score = (float)(acc + (double)noise);", ["test_oracle_local_steps.py"]),
    ("logistic_class_threshold_one_half", "(score > 0.0f ? 1.0f : 0.0f)", "(score > 0.5f ? 1.0f : 0.0f)", ["test_oracle_local_steps.py"]),
    ("minibatch_rows_share_one_word", "rows[t] = (int32_t)uniform_int(wd[t % 4], (uint32_t)s.cfg.lsq_m);",
     "rows[t] = (int32_t)uniform_int(wd[0], (uint32_t)s.cfg.lsq_m);", ["test_oracle_local_steps.py"]),
    ("write_counter_of_the_responder_not_advanced", "s.w[a] += 1; s.w[b] += 1;\n  s.pbits[a] = bits; s.pbits[b] = bits;",
     "s.w[a] += 1;\n  s.pbits[a] = bits; s.pbits[b] = bits;", ["test_oracle_interact.py"]),
    ("magnitude_rule_one_bit_short", "e = std::max(e, fm - 23);", "e = std::max(e, fm - 24);", ["test_oracle_quantizer.py"]),
    ("publish_range_from_the_maximum_alone", "lo = std::min(lo, v); hi = std::max(hi, v);\n        M = std::max(M, std::fabs(v));\n      }\n      rho = std::max(rho, hi - lo);\n    }\n    const int e = exponent_rule(rho, M, bits);",
     "hi = std::max(hi, v);\n        M = std::max(M, std::fabs(v));\n      }\n      rho = std::max(rho, hi - lo);\n    }\n    const int e = exponent_rule(rho, M, bits);",
     ["test_oracle_interact.py"]),
    ("data_matrix_scaled_by_one_over_d", "const float inv_sqrt_d = (float)(1.0 / std::sqrt((double)d));",
     "const float inv_sqrt_d = (float)(1.0 / (double)d);", ["test_oracle_local_steps.py"]),
    ("key_that_is_not_a_number_gets_cell_one", "if (std::isnan(f)) return 0;", "if (std::isnan(f)) return 1;", ["test_oracle_quantizer.py"]),
    ("saturation_dropped", "if (f >= 2147483648.0f) return std::numeric_limits<int32_t>::max();", "if (f >= 2147483648.0f) return 0;",
     ["test_oracle_quantizer.py"]),
    ("sampler_gives_up_after_four_attempts_per_pair", "attempt < 16LL * max_pairs", "attempt < 4LL * max_pairs", ["test_oracle_graph.py"]),
    ("ring_neighbours_in_the_other_order", "s.adj[(size_t)i * 2 + 0] = (i + n - 1) % n;\n      s.adj[(size_t)i * 2 + 1] = (i + 1) % n;",
     "s.adj[(size_t)i * 2 + 1] = (i + n - 1) % n;\n      s.adj[(size_t)i * 2 + 0] = (i + 1) % n;", ["test_oracle_graph.py"]),
    ("geometric_count_capped_at_three", "constexpr int kMaxGeometricTrials = 1024;", "constexpr int kMaxGeometricTrials = 3;",
     ["test_oracle_local_steps.py"]),
]


def _compile(tmp, name, text):
    src = os.path.join(tmp, name + ".cpp")
    lib = os.path.join(tmp, "lib" + name + ".so")
    with open(src, "w") as f:
        f.write(text)
    subprocess.run(["g++", "-O1", "-std=c++17", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared", "-pthread",
                    "-o", lib, src], check=True)
    return lib


def _pins_reject(lib, files):
    """True when a child pytest over the given pin files, loading `lib` as the oracle, reports a failure."""
    env = dict(os.environ, SWARM_ORACLE_LIBRARY=lib)
    cmd = [sys.executable, "-m", "pytest", "-x", "-q", "-m", "not gpu", "-p", "no:cacheprovider"]
    cmd += [os.path.join(ROOT, "tests", f) for f in files]
    r = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True)
    if r.returncode not in (0, 1):
        raise RuntimeError(f"child pytest did not run (exit {r.returncode}):\n{r.stdout[-2000:]}\n{r.stderr[-2000:]}")
    return r.returncode == 1


def test_every_planted_mistake_is_caught_by_a_pin(tmp_path):
    source = open(SOURCE).read()
    for name, old, new, _ in MUTANTS:
        assert source.count(old) == 1, f"{name}: the text to mutate must occur exactly once in the oracle source"
    all_files = sorted({f for m in MUTANTS for f in m[3]})
    jobs = [("unmutated", source, all_files)] + [(name, source.replace(old, new), files) for name, old, new, files in MUTANTS]

    def run(job):
        name, text, files = job
        return name, _pins_reject(_compile(str(tmp_path), name, text), files)

    with ThreadPoolExecutor(max(2, min(8, (os.cpu_count() or 2)))) as ex:
        results = dict(ex.map(run, jobs))
    assert results.pop("unmutated") is False, "the pins reject the oracle as it stands"
    survivors = [name for name, rejected in results.items() if not rejected]
    assert not survivors, f"no pin notices these mistakes: {survivors}"
