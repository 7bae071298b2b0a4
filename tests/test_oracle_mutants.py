"""The pins must notice a mistake.  Each case plants ONE plausible mistake in a copy of the oracle's source -- a
boundary off by one, a dropped factor, swapped operands, a wrong index -- builds it, and runs the pin tests of the
function it touches against that copy in a child process: they have to fail.  The unmodified copy has to pass.
(The mistakes are planted in the oracle, on the CPU; nothing here touches a GPU.)"""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "fd_oracle.c")

# (name, text in the source (must occur exactly once), what a mistaken author would have written, pin file)
MUTANTS = [
    ("clean_row_excludes_itself", "if (i < C) return t <= i;", "if (i < C) return t < i;", "test_oracle_attn.py"),
    ("clean_row_sees_mask_tokens", "if (i < C) return t <= i;", "if (i < C) return t <= i || t >= C;", "test_oracle_attn.py"),
    ("mask_rows_see_every_candidate", "if (t < C) return t <= r;", "if (t < C) return 1;", "test_oracle_blocks.py"),
    ("scale_dropped", "w[j] = s * p->scale;", "w[j] = s;", "test_oracle_attn.py"),
    ("k_and_v_swapped", "const uint16_t *kp = kv_ptr(p, b, j, 0, g);", "const uint16_t *kp = kv_ptr(p, b, j, 1, g);", "test_oracle_attn.py"),
    ("gqa_head_mapping", "const int g = h / (p->Hq / p->Hkv);", "const int g = h % p->Hkv;", "test_oracle_attn.py"),
    ("page_slot_transposed", "int64_t slot = j % p->page_size;", "int64_t slot = (j + 1) % p->page_size;", "test_oracle_attn.py"),
    ("softmax_not_normalised", "double pj = w[j] / den;", "double pj = w[j];", "test_oracle_attn.py"),
    ("hypothesis_off_by_one", "int r = C - nb + g;", "int r = C - nb + g + 1;", "test_oracle_blocks.py"),
    ("mask_blocks_see_each_other", "return (t - C) / kb == g;", "return 1;", "test_oracle_blocks.py"),
    ("argmax_takes_last_of_equals", "if (row[v] > row[best]) best = v;", "if (row[v] >= row[best]) best = v;", "test_oracle_accept_commit.py"),
    ("accept_compares_own_row", "while (a < k && am[a] == draft_tokens[r0 + a + 1]) ++a;", "while (a < k && am[a] == draft_tokens[r0 + a]) ++a;",
     "test_oracle_accept_commit.py"),
    ("bonus_is_the_draft", "bonus_token[b] = am[a];", "bonus_token[b] = draft_tokens[r0 + a];", "test_oracle_accept_commit.py"),
    ("commit_forgets_the_bonus", "const int new_len = n + accepted_len[b] + 1;", "const int new_len = n + accepted_len[b];", "test_oracle_accept_commit.py"),
    ("commit_keeps_a_page_too_many", "const int keep = (new_len + page_size - 1) / page_size;", "const int keep = new_len / page_size + 1;",
     "test_oracle_accept_commit.py"),
    ("accept_ratio_inverted", "if ((double)u_accept[r0 + j] * q[x] < p[x]) { ++a; continue; }", "if ((double)u_accept[r0 + j] * p[x] < q[x]) { ++a; continue; }",
     "test_oracle_accept_stochastic.py"),
    ("residual_not_clipped", "p[v] = w > 0.0 ? w : 0.0;", "p[v] = w > 0.0 ? w : -w;", "test_oracle_accept_stochastic.py"),
    ("confidence_without_bias", "double bestv = br ? (double)lr[0] + (double)br[0] : (double)lr[0];", "double bestv = (double)lr[0];",
     "test_oracle_draft_select.py"),
    ("cumulative_sum_not_product", "c *= probs[r0 + (int64_t)g * kb + u];", "c = (u ? c : 0.0) + probs[r0 + (int64_t)g * kb + u];", "test_oracle_draft_select.py"),
    ("append_starts_one_token_late", "const int j = prefix_lens[b] + i;", "const int j = prefix_lens[b] + i + 1;", "test_oracle_kv_append.py"),
    ("append_head_stride", "= v_new[(row * Hkv + h) * (int64_t)d + c];", "= v_new[(row * Hkv) * (int64_t)d + c];", "test_oracle_kv_append.py"),
    ("branch_of_the_wrong_hypothesis", "g = accepted_len[b] - (C - nb);", "g = accepted_len[b] - (C - nb) - 1;", "test_oracle_blocks.py"),
    ("bonus_drawn_at_or_below_the_target", "if (cum > target) { tok = v; break; }", "if (cum >= target * 0.5) { tok = v; break; }", "test_oracle_accept_stochastic.py"),
    ("keep_strictly_above_threshold", "if (open && c >= threshold) ++keep; else open = 0;", "if (open && c > threshold + 0.05) ++keep; else open = 0;",
     "test_oracle_draft_select.py"),
]


def _run_pins(src_path, pin_file):
    env = dict(os.environ, FD_ORACLE_SRC=src_path, OMP_NUM_THREADS="2")
    return subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "not gpu", "-p", "no:cacheprovider",
                           os.path.join(ROOT, "tests", pin_file)], cwd=ROOT, env=env, capture_output=True, text=True, timeout=900)


def test_planted_mistakes_fail_their_pins_and_the_unmodified_copy_passes(tmp_path):
    text = open(SRC).read()
    jobs = []                                                   # (name, source path, pin file, must pass?)
    control = tmp_path / "fd_oracle_copy.c"
    control.write_text(text)
    for pin_file in sorted({m[3] for m in MUTANTS}):
        jobs.append(("unmodified:" + pin_file, str(control), pin_file, True))
    for name, old, new, pin_file in MUTANTS:
        assert text.count(old) == 1, f"{name}: the text to replace must occur exactly once in the oracle's source"
        path = tmp_path / f"fd_oracle_{name}.c"
        path.write_text(text.replace(old, new))
        jobs.append((name, str(path), pin_file, False))
    # the copy is built once, before the children share it
    subprocess.run(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", str(control) + ".so", str(control), "-lm"], check=True)
    with ThreadPoolExecutor(max_workers=max(1, min(8, (os.cpu_count() or 2) // 2))) as pool:
        results = list(pool.map(lambda j: _run_pins(j[1], j[2]), jobs))
    unnoticed, broken = [], []
    for (name, _, pin_file, must_pass), r in zip(jobs, results):
        if must_pass:
            if r.returncode != 0:
                broken.append((name, r.stdout[-1500:]))
        elif r.returncode == 0:
            unnoticed.append(f"{name} ({pin_file})")
        elif " failed" not in r.stdout:                          # the pins have to FAIL, not fail to build or to collect
            broken.append((name, r.stdout[-1500:] + r.stderr[-500:]))
    assert not broken, broken
    assert not unnoticed, f"no pin noticed: {unnoticed}"
