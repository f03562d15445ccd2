"""Are the oracle's pins sharp?  Each case plants one plausible mistake in a COPY of the oracle's
source (on the CPU; the real oracle is untouched), compiles it and runs the pin tests against
the broken copy: at least one pin must fail."""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
PINS = ["tests/test_oracle_philox.py", "tests/test_oracle_sampler.py",
        "tests/test_oracle_perturb.py", "tests/test_oracle_adagrad.py", "tests/test_oracle_sync.py"]

# (name, text in oracle/gbmuf_oracle.cpp, replacement)
MUTANTS = [
    ("philox_multipliers_swapped", "M0 = 0xD2511F53ull, M1 = 0xCD9E8D57ull",
     "M0 = 0xCD9E8D57ull, M1 = 0xD2511F53ull"),
    ("philox_nine_rounds", "for (int r = 0; r < 10; ++r) {", "for (int r = 0; r < 9; ++r) {"),
    ("philox_key_not_bumped", "if (r > 0) { key0 += W0; key1 += W1; }", ""),
    ("philox_outputs_transposed", "nxt.w[1] = (uint32_t)p1;", "nxt.w[1] = (uint32_t)p0;"),
    ("ring_only_forward", "int64_t raw = side == 0 ? (int64_t)k - d : (int64_t)k + d;",
     "int64_t raw = (int64_t)k + d + (side == 0 ? p : 0);"),
    ("ring_order_swapped", "int64_t raw = side == 0 ? (int64_t)k - d : (int64_t)k + d;",
     "int64_t raw = side == 1 ? (int64_t)k - d : (int64_t)k + d;"),
    ("sampler_with_replacement", "const int32_t tmp = a[j]; a[j] = a[t]; a[t] = tmp;",
     "const int32_t tmp = a[t]; a[t] = a[j]; a[j] = tmp; a[t] = tmp;"),
    ("sampler_range_not_shrinking", "(uint64_t)(c - j)) >> 32)", "(uint64_t)(c - j - (j > 0))) >> 32)"),
    ("sampler_ignores_component", "(uint32_t)(comp_base + i),", "(uint32_t)(comp_base),"),
    ("sampler_ignores_round_hi", "(uint32_t)(round >> 32), (uint32_t)(comp_base + i)",
     "0u, (uint32_t)(comp_base + i)"),
    ("sampler_reuses_word", "const uint32_t u = rnd.w[j % 4];", "const uint32_t u = rnd.w[0];"),
    ("avg_divides_by_q", "const float avg = s / (float)(q + 1);",
     "const float avg = s / (float)(q > 0 ? q : 1);"),
    ("avg_drops_own_value", "float s = load_theta(S, dtype, at);", "float s = 0.0f;"),
    ("avg_reads_updated_replicas", "s = s + load_theta(S, dtype, (int64_t)nb[j] * ld + e);",
     "s = s + load_theta(theta, dtype, (int64_t)nb[j] * ld + e);"),
    ("avg_reads_own_row_for_neighbours", "(int64_t)nb[j] * ld + e);", "(int64_t)k * ld + e);"),
    ("block_delta_sign", "const float g = avg - load_theta(rst, dtype, at);",
     "const float g = load_theta(rst, dtype, at) - avg;"),
    ("block_delta_against_current_theta", "const float g = avg - load_theta(rst, dtype, at);",
     "const float g = avg - load_theta(S, dtype, at);"),
    ("momentum_term_dropped", "const float d = md + zg;", "const float d = zg;"),
    ("momentum_zeta_dropped", "const float zg = zeta * g;", "const float zg = g;"),
    ("momentum_eta_on_g", "const float md = eta * delta[at];", "const float md = delta[at];"),
    ("omega_adds_g", "const float w = omega[at] + d;", "const float w = omega[at] + g;"),
    ("restart_without_eta", "const float nd = eta * d;", "const float nd = d;"),
    ("restart_without_lookahead", "const float t = w + nd;", "const float t = w;"),
    ("block_start_not_refreshed", "store_theta(rst, dtype, at, stored);", ""),
    ("ma_mode_falls_through", "if (mode == 1) {", "if (mode == 7) {"),
    ("sync_flags_ignored", "if (sync && !sync[i]) continue;", ""),
    ("bf16_truncates", "u += 0x7FFFu + lsb;", ""),
    ("bf16_rounds_half_up", "u += 0x7FFFu + lsb;", "u += 0x8000u;"),
    ("perturb_sign", "v = v - upd;", "v = v + upd;"),
    ("perturb_pair_shares_words", "const uint32_t a = (ge & 1) ? r.w[2] : r.w[0];",
     "const uint32_t a = r.w[0];"),
    ("perturb_not_centred", "(float)(sum - 131070) * C", "(float)(sum - 131072) * C"),
    ("perturb_ignores_worker", "(uint32_t)(pair >> 32), (uint32_t)k, (uint32_t)(step + s)",
     "(uint32_t)(pair >> 32), 0u, (uint32_t)(step + s)"),
    ("perturb_local_index", "const uint64_t ge = (uint64_t)(elem_base + e);",
     "const uint64_t ge = (uint64_t)(e);"),
    ("adagrad_accumulates_unclipped", "const float gg = g * g;", "const float gg = grad[at] * grad[at];"),
    ("adagrad_no_sqrt", "const float denom = std::sqrt(a) + eps;", "const float denom = a + eps;"),
    ("adagrad_sign", "load_theta(theta, dtype, at) - upd);", "load_theta(theta, dtype, at) + upd);"),
    ("adagrad_lr_dropped", "const float num = lr * g;", "const float num = g;"),
    ("adagrad_clip_inverted", "scale = clip_norm / (norm > clip_norm ? norm : clip_norm);",
     "scale = (norm > clip_norm ? norm : clip_norm) / clip_norm;"),
    ("adagrad_clips_always", "scale = clip_norm / (norm > clip_norm ? norm : clip_norm);",
     "scale = clip_norm / norm;"),
    ("adagrad_norm_over_everything", "for (int64_t e = ranges[2 * r]; e < ranges[2 * r + 1]; ++e) {",
     "for (int64_t e = 0; e < N; ++e) {"),
    ("adagrad_scales_outside_ranges", "if (inside && clip_norm > 0.0f) g = g * scale;",
     "if (clip_norm > 0.0f) g = g * scale;"),
    ("adagrad_accumulator_not_stored", "accum[at] = a;", ""),
    ("final_average_divides_by_k_minus_1", "s / (float)K", "s / (float)(K > 1 ? K - 1 : 1)"),
]


def _run_mutant(args):
    name, old, new, tmp = args
    import oracle
    src = open(os.path.join(ROOT, "oracle", "gbmuf_oracle.cpp")).read()
    assert src.count(old) == 1, f"{name}: the text to mutate must occur exactly once"
    cpp = os.path.join(tmp, name + ".cpp")
    so = os.path.join(tmp, name + ".so")
    with open(cpp, "w") as f:
        f.write(src.replace(old, new))
    subprocess.run(["g++", *oracle.CXXFLAGS, cpp, "-o", so], check=True)
    env = dict(os.environ, GBMUF_ORACLE_LIB=so)
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                        *PINS], cwd=ROOT, env=env, capture_output=True, text=True)
    return name, r.returncode, r.stdout[-400:]


def test_every_planted_mistake_is_caught(tmp_path):
    jobs = [(n, o, r, str(tmp_path)) for n, o, r in MUTANTS]
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 2)) as ex:
        results = list(ex.map(_run_mutant, jobs))
    survivors = [n for n, rc, _ in results if rc == 0]
    broken_runs = [(n, out) for n, rc, out in results if rc not in (0, 1)]
    assert not broken_runs, broken_runs
    assert not survivors, f"pins did not notice: {survivors}"
